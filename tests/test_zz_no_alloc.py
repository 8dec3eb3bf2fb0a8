"""The allocation-free entry point, dyspec_tree_attention_static, against dyspec_tree_attention_ragged
and against the fp64 oracle.

For callers that cannot allocate device memory (everything was given to a pool at start-up, or the
host framework forbids allocation inside its step function) the library keeps the work list and the
split-KV partials in a fixed 16 MiB device array.  The array is shared and keeps old contents, so
the check runs two calls back to back, of different shapes, and each must match the ordinary entry
point and, element by element, the oracle (same tolerance as the parity tests).  It also checks what
the entry point exists for: the device's free memory does not change across calls of new shapes.
This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest

from paper_2410_11744_b200 import workloads as wl

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3       # the tolerance of the parity tests


def _bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def test_static_scratch_entry_point_matches_ragged_entry_point_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding as B, runner as R

    # the first case is cut into split-KV pieces (about 12 MiB of partials in the scratch array); the
    # cases after it are smaller and of other shapes (config 2 merges its splits on chip and only
    # needs the work list), so stale contents would show; then the first shape again
    rng = np.random.default_rng(3)
    big = wl.make_custom(20, 64, 8, 128, [1500], [wl.greedy_tree(rng, 40, 8, 0.3)])
    # ... and one request with more (kv head, query tile) groups than CTAs: through a plan it runs from
    # the shared queue in the caller's workspace, here (no workspace) from fixed lists
    many = wl.make_custom(22, 64, 8, 128, [200], [wl.greedy_tree(rng, 1024, 8, 0.3)])
    # ... and a shape that runs as one thread-block cluster per group in the tensor-core regime (its CTAs' shares
    # of the partials go through the scratch array, 7.5 MiB here)
    clustered = wl.make_custom(23, 8, 8, 128, [2000], [wl.greedy_tree(rng, 256, 8, 0.3)])
    cases = [big, wl.make_custom(21, 8, 2, 64, [300], [wl.greedy_tree(rng, 40, 4, 0.3)]), wl.make_config(2), many,
             clustered, big]
    from oracle import dyspec_oracle as orc
    for w in cases:
        batch = R.DeviceBatch(w)
        batch.step()                                          # existing entry points: mask + ragged attention
        bits, _, want_bits, status = batch.results()
        assert status == 0
        assert batch.plan.describe()["dynamic"] == (1 if w is many else 0)
        if w is clustered:
            assert batch.plan.describe()["regime"] == 1 and batch.plan.describe()["cluster"] == 8
        L, n = int(w.prefix_len[0]), int(w.n_nodes[0])
        out = torch.zeros_like(batch.out)
        st = torch.zeros((1,), dtype=torch.int32, device=out.device)
        for _ in range(2):                                    # two calls in a row on the shared array
            out.zero_()
            B.dyspec_tree_attention_static(batch.q, batch.k, batch.v, L, batch.bits, n, out, w.n_q_heads,
                                           w.n_kv_heads, w.head_dim, batch.W, 0.0, st)
            torch.cuda.synchronize()
            assert int(st.item()) == 0
            got = _bits_to_f64(R.bf16_tensor_to_bits(out))
            want = _bits_to_f64(want_bits)
            assert np.isfinite(got).all()
            err = np.abs(got - want)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
        # the last call's output against the definition (fp64 oracle), element by element
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        err = np.abs(got - ref)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (w.name, err.max(), err.mean())


def test_static_entry_point_allocates_no_device_memory():
    """Calls of shapes never seen before leave the driver's free-memory figure unchanged (all buffers are
    made beforehand; the entry point itself must not allocate), and a request with no nodes is a no-op."""
    import torch
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding as B, runner as R
    rng = np.random.default_rng(5)
    shapes = [(8, 2, 64, 90, 17), (32, 32, 128, 700, 48), (64, 8, 128, 333, 300), (16, 4, 128, 0, 5)]
    batches = []
    for i, (hq, hkv, d, L, n) in enumerate(shapes):
        w = wl.make_custom(40 + i, hq, hkv, d, [L], [wl.greedy_tree(rng, n, 4, 0.3)])
        b = R.DeviceBatch(w)
        b.build_mask()
        batches.append((w, b, torch.zeros_like(b.out)))
    # warm-up call: the first call on a device looks up the array's address and loads the kernels
    w, b, out = batches[0]
    B.dyspec_tree_attention_static(b.q, b.k, b.v, int(w.prefix_len[0]), b.bits, int(w.n_nodes[0]), out, w.n_q_heads,
                                   w.n_kv_heads, w.head_dim, b.W)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for w, b, out in batches[1:] + batches[:1]:
        B.dyspec_tree_attention_static(b.q, b.k, b.v, int(w.prefix_len[0]), b.bits, int(w.n_nodes[0]), out, w.n_q_heads,
                                       w.n_kv_heads, w.head_dim, b.W)
        # no nodes: returns at once, touches nothing
        B.dyspec_tree_attention_static(b.q, b.k, b.v, int(w.prefix_len[0]), b.bits, 0, out, w.n_q_heads, w.n_kv_heads,
                                       w.head_dim, b.W)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    for w, b, out in batches:
        assert out.any()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    import torch
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding as B, runner as R
    # 32 heads x 5 splits merged through the workspace: ~21 MiB of partials, over the 16 MiB array.  (The plan the
    # scheduler would choose by itself for this shape is a cluster plan, which needs no workspace at all: the
    # workspace merge is asked for here.)
    w = wl.make_config(3)
    batch = R.DeviceBatch(w)
    batch.build_mask()
    out = torch.zeros_like(batch.out)
    B.dyspec_set_tuning(-1, 0, 1)
    try:
        with pytest.raises(B.DyspecError) as e:
            B.dyspec_tree_attention_static(batch.q, batch.k, batch.v, int(w.prefix_len[0]), batch.bits, int(w.n_nodes[0]),
                                           out, w.n_q_heads, w.n_kv_heads, w.head_dim, batch.W)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    assert e.value.code == -3
    torch.cuda.synchronize()
    assert not out.any()
