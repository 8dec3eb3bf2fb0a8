"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by element.

Masks and depths must match bit-exactly.  Attention: bf16 inputs, fp32 accumulation, bf16 output,
compared with the fp64 oracle: max abs error <= 2e-2 and mean abs error <= 2e-3.
"""
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


def run_and_check(rt, w, regime=-1, ctas=0, words_per_row=None, fuse=2):
    B, R = rt
    B.dyspec_set_tuning(regime, ctas, fuse)
    try:
        batch = R.DeviceBatch(w, words_per_row=words_per_row)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    batch.step()
    bits, depths, out_bits, status = batch.results()
    assert status == 0
    ref_bits, ref_depths = orc.build_tree_mask_ragged(w.parents, batch.W)
    assert np.array_equal(bits, ref_bits)
    assert np.array_equal(depths, ref_depths)
    ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
    got = orc.bf16_bits_to_f64(out_bits)
    assert np.isfinite(got).all()
    if ref.size:
        err = np.abs(got - ref)
        assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
        assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    return batch, got, ref


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_configs_match_oracle(rt, index):
    run_and_check(rt, wl.make_config(index))


@pytest.mark.parametrize("case", ["one_tile", "two_halves", "multi_tile", "c3", "c4", "c5"])
def test_tensor_core_regime(rt, case):
    """The tcgen05 kernel (regime 1) forced on: single tile first, then both query halves, long key loops, configs."""
    rng = np.random.default_rng(5)
    if case == "one_tile":
        w = wl.make_custom(40, 8, 1, 128, [100], [wl.greedy_tree(rng, 16, 4, 0.3)])        # 128 rows, 2 key tiles
    elif case == "two_halves":
        w = wl.make_custom(41, 8, 1, 128, [128], [wl.greedy_tree(rng, 32, 4, 0.3)])        # 256 rows
    elif case == "multi_tile":
        w = wl.make_custom(42, 16, 2, 128, [1500, 300], [wl.greedy_tree(rng, 200, 8, 0.2), wl.chain_tree(70)])
    else:
        w = wl.make_config(int(case[1]))
    run_and_check(rt, w, regime=1)


@pytest.mark.parametrize("hq,hkv,d", [(8, 1, 64), (4, 4, 64), (4, 4, 128), (4, 2, 128)])
def test_tensor_core_regime_shapes(rt, hq, hkv, d):
    rng = np.random.default_rng(hq * 10 + d)
    trees = [wl.greedy_tree(rng, 300, 8, 0.3), wl.random_tree(rng, 130, 0.05), np.zeros(0, np.int32), wl.chain_tree(129)]
    for ctas in (0, 5):
        run_and_check(rt, wl.make_custom(15, hq, hkv, d, [260, 64, 3, 0], trees), regime=1, ctas=ctas)


@pytest.mark.parametrize("hq,hkv,d,L,n", [(32, 32, 128, 1024, 64), (16, 16, 64, 700, 40), (8, 2, 128, 3000, 16),
                                          (4, 4, 128, 9000, 33), (64, 8, 128, 600, 8)])
def test_cluster_combine(rt, hq, hkv, d, L, n):
    """Uniform small batches: one thread-block cluster per query tile, partials merged through
    distributed shared memory (cluster sizes 2, 4 and 8, both head dims, ragged last rows)."""
    B, _ = rt
    rng = np.random.default_rng(hq + n)
    w = wl.make_custom(50, hq, hkv, d, [L], [wl.greedy_tree(rng, n, 4, 0.3)])
    batch, _, _ = run_and_check(rt, w)
    assert batch.plan.describe()["cluster"] > 1


@pytest.mark.parametrize("fuse", [0, 2])
@pytest.mark.parametrize("ctas", [1, 3, 40, 1000])
def test_split_count_does_not_change_results(rt, ctas, fuse):
    """Forcing the scheduler to balance over few or many CTAs changes the split-KV cuts, not the answer."""
    w = wl.make_custom(77, 8, 2, 128, [700, 45], [wl.greedy_tree(np.random.default_rng(1), 90, 8, 0.3),
                                                   wl.greedy_tree(np.random.default_rng(2), 33, 4, 0.2)])
    _, got, _ = run_and_check(rt, w, ctas=ctas, fuse=fuse)
    _, base, _ = run_and_check(rt, w, ctas=2)
    assert np.abs(got - base).max() <= 2 ** -6     # both are bf16 roundings of nearly equal fp32 values


@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 64), (8, 4, 64), (8, 2, 128), (8, 1, 128), (2, 2, 128)])
def test_shapes_and_gqa(rt, hq, hkv, d):
    rng = np.random.default_rng(hq * 100 + d)
    trees = [wl.greedy_tree(rng, 37, 4, 0.3), wl.random_tree(rng, 130, 0.05), wl.chain_tree(65)]
    run_and_check(rt, wl.make_custom(5, hq, hkv, d, [129, 64, 1], trees))


def test_edge_cases(rt):
    rng = np.random.default_rng(0)
    # empty prefix; single node; an empty request in the middle; star forest; ragged tails
    trees = [wl.chain_tree(5), np.zeros(0, np.int32), wl.star_forest(70), np.array([-1], np.int32),
             wl.greedy_tree(rng, 63, 4, 0.3)]
    run_and_check(rt, wl.make_custom(6, 4, 2, 64, [0, 10, 63, 0, 65], trees))
    # nothing at all
    run_and_check(rt, wl.make_custom(7, 4, 4, 64, [], []))
    run_and_check(rt, wl.make_custom(8, 4, 4, 64, [5], [np.zeros(0, np.int32)]))


def test_maximum_tree_size(rt):
    rng = np.random.default_rng(4)
    w = wl.make_custom(9, 8, 1, 128, [100], [wl.greedy_tree(rng, 1024, 8, 0.2)])
    run_and_check(rt, w)
    w = wl.make_custom(10, 2, 2, 64, [3], [wl.chain_tree(1024)])          # depth 1023: deepest possible
    run_and_check(rt, w)


def test_rows_after_a_request_may_hold_garbage(rt):
    """K/V rows that follow a request (another request's, or unwritten memory) must not leak in, even as NaN."""
    rng = np.random.default_rng(11)
    trees = [wl.greedy_tree(rng, 20, 4, 0.3), wl.greedy_tree(rng, 9, 4, 0.3)]
    w = wl.make_custom(12, 4, 2, 128, [70, 30], trees)
    # poison request 1's rows as seen from request 0's last tiles, then restore them for request 1 by
    # putting a gap of NaN rows between the two requests instead
    gap = 100
    nan_rows = np.full((gap,) + w.k.shape[1:], 0x7FC0, dtype=np.uint16)
    o1 = int(w.kv_row_offset[1])
    w.k = np.concatenate([w.k[:o1], nan_rows, w.k[o1:], nan_rows])
    w.v = np.concatenate([w.v[:o1], nan_rows, w.v[o1:], nan_rows])
    w.kv_row_offset = np.array([0, o1 + gap], dtype=np.int64)
    run_and_check(rt, w)


def test_bad_tree_is_reported_not_fatal(rt):
    import torch
    B, R = rt
    w = wl.make_custom(13, 4, 4, 64, [16], [np.array([-1, 0, 5, 1, -3, 2], np.int32)])   # nodes 2 and 4 are bad
    batch = R.DeviceBatch(w)
    batch.step()
    bits, depths, out_bits, status = batch.results()
    assert status == -5
    fixed = [-1, 0, -1, 1, -1, 2]                 # bad nodes become roots
    ref_bits, ref_depths = orc.build_tree_mask(fixed, batch.W)
    assert np.array_equal(bits, ref_bits) and np.array_equal(depths, ref_depths)
    assert np.isfinite(orc.bf16_bits_to_f64(out_bits)).all()


def test_single_request_entry_points(rt):
    import torch
    B, R = rt
    w = wl.make_config(1)
    L, n = int(w.prefix_len[0]), int(w.n_nodes[0])
    W = B.dyspec_words_per_row(n)
    dev = torch.device("cuda:0")
    parents = torch.from_numpy(w.parents[0]).to(dev)
    bits = torch.zeros((n, W), dtype=torch.int32, device=dev)
    depths = torch.zeros((n,), dtype=torch.int32, device=dev)
    B.dyspec_build_tree_mask(parents, n, bits, depths, W)
    q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
    k = torch.from_numpy(w.k.view(np.int16)).to(dev).view(torch.bfloat16)
    v = torch.from_numpy(w.v.view(np.int16)).to(dev).view(torch.bfloat16)
    out = torch.zeros_like(q)
    B.dyspec_set_default_shape(w.n_q_heads, w.n_kv_heads, w.head_dim, W, 0.0)
    for _ in range(2):                               # second call reuses the cached plan
        out.zero_()
        B.dyspec_tree_attention(q, k, v, L, bits, n, out)
        torch.cuda.synchronize()
        ref_bits, ref_depths = orc.build_tree_mask(w.parents[0], W)
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), ref_bits)
        assert np.array_equal(depths.cpu().numpy(), ref_depths)
        got = orc.bf16_bits_to_f64(R.bf16_tensor_to_bits(out))
        ref = orc.tree_attention(w.q, w.k, w.v, L, w.parents[0])
        assert np.abs(got - ref).max() <= MAX_ABS and np.abs(got - ref).mean() <= MEAN_ABS


def test_single_request_form_follows_a_change_of_scale(rt):
    """The cached plans of the convenience form are keyed by the scale too: the same shape with another
    scale must not reuse the old plan."""
    import torch
    B, R = rt
    w = wl.make_config(1)
    L, n = int(w.prefix_len[0]), int(w.n_nodes[0])
    W = B.dyspec_words_per_row(n)
    dev = torch.device("cuda:0")
    parents = torch.from_numpy(w.parents[0]).to(dev)
    bits = torch.zeros((n, W), dtype=torch.int32, device=dev)
    depths = torch.zeros((n,), dtype=torch.int32, device=dev)
    B.dyspec_build_tree_mask(parents, n, bits, depths, W)
    q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
    k = torch.from_numpy(w.k.view(np.int16)).to(dev).view(torch.bfloat16)
    v = torch.from_numpy(w.v.view(np.int16)).to(dev).view(torch.bfloat16)
    out = torch.zeros_like(q)
    for scale in (0.05, 0.3, 0.05):
        B.dyspec_set_default_shape(w.n_q_heads, w.n_kv_heads, w.head_dim, W, scale)
        out.zero_()
        B.dyspec_tree_attention(q, k, v, L, bits, n, out)
        torch.cuda.synchronize()
        got = orc.bf16_bits_to_f64(R.bf16_tensor_to_bits(out))
        ref = orc.tree_attention(w.q, w.k, w.v, L, w.parents[0], scale=scale)
        assert np.abs(got - ref).max() <= MAX_ABS and np.abs(got - ref).mean() <= MEAN_ABS, scale


def test_runs_are_bitwise_repeatable(rt):
    """Also checks that the arrival counters of the fused combine are left at zero by every call."""
    w = wl.make_config(2)
    batch, got, _ = run_and_check(rt, w)
    first = batch.results()[2].copy()
    for _ in range(3):
        batch.out.zero_()
        batch.step()
        assert np.array_equal(batch.results()[2], first)


def test_shared_queue_plan_is_repeatable_and_leaves_the_queue_empty(rt):
    """More groups than CTAs in the tensor-core regime: the CTAs take whole groups from a shared queue.
    Every launch must see the queue as the previous one left it (cleared), back to back and through
    two buffer sets that share the plan, and the result cannot depend on which CTA took which group."""
    B, R = rt
    rng = np.random.default_rng(31)
    trees = [wl.greedy_tree(rng, n, 8, 0.3) for n in (300, 700, 130, 520)]
    w = wl.make_custom(33, 16, 2, 128, [600, 90, 2000, 0], trees)      # 8 rows per node: 52 query tiles x 2 kv heads... x 4 requests
    w_big = wl.make_custom(34, 64, 8, 128, [1500, 300, 40, 700, 2500, 0], [wl.greedy_tree(rng, n, 8, 0.3) for n in (400, 640, 96, 512, 333, 768)])
    w_d64 = wl.make_custom(35, 32, 8, 64, [900, 64, 0, 1300, 257], [wl.greedy_tree(rng, n, 8, 0.3) for n in (700, 512, 90, 640, 333)])
    for wk in (w, w_big, w_d64):
        batch, got, _ = run_and_check(rt, wk, regime=1)
        info = batch.plan.describe()
        if wk is not w:
            assert info["dynamic"] == 1 and info["split_groups"] == 0 and info["groups"] > info["ctas"]
        first = batch.results()[2].copy()
        twin = R.DeviceBatch(wk, plan=batch.plan)
        for _ in range(3):
            batch.out.zero_()
            batch.step()
            twin.step()
            assert np.array_equal(batch.results()[2], first)
            assert np.array_equal(twin.results()[2], first)
    # the budgeted split plan (fixed lists, partials merged by the combine kernel) agrees up to the
    # rounding of a different summation order
    B.dyspec_set_tuning(1, 0, 2 + 16)
    try:
        fixed = R.DeviceBatch(w_big)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    assert fixed.plan.describe()["dynamic"] == 0
    fixed.step()
    first = R.DeviceBatch(w_big)
    first.step()
    first = first.results()[2]
    diff = np.abs(orc.bf16_bits_to_f64(fixed.results()[2]) - orc.bf16_bits_to_f64(first))
    assert diff.max() <= MAX_ABS


def test_mask_builder_batched_without_a_plan(rt):
    """dyspec_build_tree_mask_batched (host node offsets, no plan) == the oracle, request by request,
    including an empty request and a bad parent that must be reported for its own request only."""
    import torch
    B, _ = rt
    rng = np.random.default_rng(41)
    trees = [wl.greedy_tree(rng, 70, 6, 0.3), np.zeros(0, np.int32), wl.chain_tree(5), wl.random_tree(rng, 300),
             np.array([-1, 0, 7, 1], np.int32)]                       # entry 2 of the last tree is invalid
    offs = np.concatenate([[0], np.cumsum([len(t) for t in trees])]).astype(np.int32)
    n = int(offs[-1])
    W = B.dyspec_words_per_row(max(len(t) for t in trees))
    dev = "cuda:0"
    parents = torch.from_numpy(np.concatenate(trees).astype(np.int32)).to(dev)
    bits = torch.full((n, W), -1, dtype=torch.int32, device=dev)
    depths = torch.full((n,), -1, dtype=torch.int32, device=dev)
    status = torch.zeros(len(trees), dtype=torch.int32, device=dev)
    B.dyspec_build_tree_mask_batched(parents, offs.tolist(), bits, depths, W, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy().tolist() == [0, 0, 0, 0, -5]
    fixed = [t.copy() for t in trees]
    fixed[-1][2] = -1                                                   # an invalid parent is treated as "no parent"
    ref_bits, ref_depths = orc.build_tree_mask_ragged(fixed, W)
    assert np.array_equal(bits.cpu().numpy().view(np.uint32), ref_bits)
    assert np.array_equal(depths.cpu().numpy(), ref_depths)
    with pytest.raises(B.DyspecError):
        B.dyspec_build_tree_mask_batched(parents, [0, 5, 3], bits, depths, W, None)     # offsets must not decrease


@pytest.mark.parametrize("hq,hkv,n,L", [(4, 4, 40, 500), (8, 1, 8, 700), (16, 2, 100, 600), (32, 32, 64, 1024)])
def test_growing_maxima_exercise_the_lazy_rescale(rt, hq, hkv, n, L):
    """Keys whose scores grow steadily along the sequence (by tens of log2 units in all): both kernels keep
    their running output in tensor memory against a lazy reference and rescale it only when a row maximum
    has grown by more than 2^8, which random N(0,1) inputs never do.  Here they must, several times."""
    rng = np.random.default_rng(hq * 1000 + n)
    w = wl.make_custom(70 + n, hq, hkv, 128, [L], [wl.greedy_tree(rng, n, 6, 0.3)])
    pattern = np.where(rng.random(128) < 0.5, -1.0, 1.0)
    q = pattern[None, None, :] * (1.0 + 0.1 * rng.standard_normal((n, hq, 1))) + 0.05 * rng.standard_normal((n, hq, 128))
    rows = w.k.shape[0]
    ramp = (0.02 + 2.0 * np.arange(rows) / rows)[:, None, None]           # |score| grows ~ 30 log2 units over the cache
    k = pattern[None, None, :] * ramp + 0.05 * rng.standard_normal((rows, hkv, 128))
    def to_bits(x):
        u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
        return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    w.q[...] = to_bits(q)
    w.k[...] = to_bits(k)
    for regime in (0, 1) if n * (hq // hkv) <= 64 else (1,):
        run_and_check(rt, w, regime=regime)
    run_and_check(rt, w)


@pytest.mark.parametrize("n_nodes,heads", [(64, (8, 8)), (48, (32, 4)), (1024, (2, 2))])
def test_mask_of_this_step_is_the_one_used_when_the_tree_changes(rt, n_nodes, heads):
    """The attention kernels start on the prefix tiles before the mask builder of the same step has
    finished and wait for it only in front of the tree tiles.  Same buffers, same shape, the tree
    changes from step to step (chain, star, random): a mask word read too early would be the previous
    step's."""
    import torch
    B, R = rt
    rng = np.random.default_rng(n_nodes)
    trees = [wl.chain_tree(n_nodes), wl.star_forest(n_nodes), wl.random_tree(rng, n_nodes), wl.chain_tree(n_nodes)]
    ws = [wl.make_custom(77, heads[0], heads[1], 64, [200], [t]) for t in trees]      # same seed: same Q, K, V
    batch = R.DeviceBatch(ws[0])
    refs = [orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents) for w in ws]
    for it in range(12):
        k = it % len(ws)
        batch.parents.copy_(torch.from_numpy(ws[k].parents_concat).to(batch.parents.device))
        batch.step()
        bits, depths, out_bits, status = batch.results()
        assert status == 0
        ref_bits, _ = orc.build_tree_mask_ragged(ws[k].parents, batch.W)
        assert np.array_equal(bits, ref_bits)
        err = np.abs(orc.bf16_bits_to_f64(out_bits) - refs[k])
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (it, k, err.max())


@pytest.mark.parametrize("shape", ["split_small_tiles", "split_tensor_core"])
def test_calls_that_follow_each_other_may_share_a_workspace(rt, shape):
    """Split-KV plans (partials + combine launch): two batches with different inputs share ONE plan and
    ONE workspace and are stepped alternately without any synchronisation in between.  The kernels of
    consecutive calls overlap on the GPU (early start), so a call that wrote its partials before the
    previous call's combine had read its own would corrupt the previous output."""
    B, R = rt
    if shape == "split_small_tiles":
        mk = lambda seed: wl.make_custom(seed, 8, 8, 128, [3000, 700], [wl.greedy_tree(np.random.default_rng(5), 48, 4, 0.3),
                                                                      wl.chain_tree(17)])
        tuning = (-1, 0, 0)          # separate combine kernel instead of the cluster merge
    else:
        mk = lambda seed: wl.make_custom(seed, 4, 4, 128, [2500], [wl.random_tree(np.random.default_rng(6), 256)])
        tuning = (-1, 0, 1)          # merged inside the kernel through the workspace (the default plan for this shape
                                     # is a cluster plan, which has no workspace)
    wa, wb = mk(301), mk(302)
    B.dyspec_set_tuning(*tuning)
    try:
        ba = R.DeviceBatch(wa)
        bb = R.DeviceBatch(wb, plan=ba.plan)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    assert ba.plan.describe()["split_groups"] > 0
    bb.workspace, bb.workspace_bytes = ba.workspace, ba.workspace_bytes
    for _ in range(6):
        ba.step()
        bb.step()
    for batch, w in ((ba, wa), (bb, wb)):
        bits, depths, out_bits, status = batch.results()
        assert status == 0
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        err = np.abs(orc.bf16_bits_to_f64(out_bits) - ref)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (shape, err.max())


@pytest.mark.parametrize("hq,hkv,d,L,n,ctas", [(8, 1, 128, 20000, 40, 0), (8, 1, 64, 9000, 40, 0), (4, 4, 128, 3000, 300, 37),
                                               (16, 2, 64, 700, 260, 11)])
def test_merge_inside_the_tensor_core_kernel(rt, hq, hkv, d, L, n, ctas):
    """Split-KV groups of the tensor-core regime are merged by their own items (no combine launch): few
    groups cut into many equal pieces, one per CTA (more than eight splits, so the merge walks the
    partials in several rounds; both head dimensions), and forced CTA counts that give CTAs several split
    items of different groups.  The counters in the workspace must be back at zero: a second call on the
    same buffers gives the same bits."""
    B, R = rt
    rng = np.random.default_rng(hq * 1000 + n)
    w = wl.make_custom(70, hq, hkv, d, [L], [wl.greedy_tree(rng, n, 6, 0.3)])
    batch, got, _ = run_and_check(rt, w, regime=1, ctas=ctas, fuse=1 + (16 if ctas else 0))     # 1: never clusters
    info = batch.plan.describe()
    assert info["regime"] == 1 and info["split_groups"] > 0 and info["combine_launch"] == 0 and info["cluster"] == 1
    if ctas == 0:
        assert info["max_splits"] > 8 or d == 64
    batch.out.zero_()
    batch.attention()
    _, _, out2, status = batch.results()
    assert status == 0 and np.array_equal(orc.bf16_bits_to_f64(out2), got)


@pytest.mark.parametrize("hq,hkv,d,L,n,want_c", [(8, 8, 128, 2000, 256, 8), (16, 16, 128, 1500, 200, 4), (64, 64, 64, 700, 130, 2),
                                                 (8, 1, 128, 3000, 12, 8), (32, 4, 64, 1000, 64, 4)])
def test_cluster_merge_in_the_tensor_core_regime(rt, hq, hkv, d, L, n, want_c):
    """Few groups of equal length: one thread-block cluster per group, every CTA merges its share of the rows
    once the cluster's barrier says that all partials are written.  Cluster sizes 2, 4 and 8, both head dimensions,
    a ragged second half, a group with one half only (the other half parks neutral rows), GQA.  No second
    launch, no counters; a second call on the same buffers gives the same bits."""
    B, R = rt
    rng = np.random.default_rng(hq * 100 + n)
    w = wl.make_custom(75, hq, hkv, d, [L], [wl.greedy_tree(rng, n, 6, 0.3)])
    batch, got, _ = run_and_check(rt, w, regime=1)
    info = batch.plan.describe()
    assert info["regime"] == 1 and info["cluster"] == want_c and info["combine_launch"] == 0, info
    assert batch.plan.workspace_bytes() > 0                          # the peers' shares travel through the workspace
    batch.out.zero_()
    batch.attention()
    _, _, out2, status = batch.results()
    assert status == 0 and np.array_equal(orc.bf16_bits_to_f64(out2), got)
    # the same request merged through the workspace instead: the same result up to the order of the additions
    _, got_l2, _ = run_and_check(rt, w, regime=1, fuse=1)
    assert np.abs(got_l2 - got).max() <= 2e-2
