"""GPU parity of the accepted-path KV compaction with the oracle (bit exact), alone and chained behind
the verification kernel."""
import numpy as np
import pytest

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding
    return binding


@pytest.mark.parametrize("keep_root", [False, True])
@pytest.mark.parametrize("hkv,d", [(8, 128), (32, 128), (1, 64), (2, 8)])
def test_compact_matches_oracle(B, hkv, d, keep_root):
    import torch
    rng = np.random.default_rng(hkv * 100 + d)
    n_req, max_out = 6, 16
    Ls = rng.integers(0, 40, size=n_req)
    ns = rng.integers(1, 50, size=n_req)
    offs = np.concatenate([[0], np.cumsum(Ls + ns)[:-1]]).astype(np.int64)
    rows = int((Ls + ns).sum()) + 3
    k = rng.integers(0, 65536, size=(rows, hkv, d), dtype=np.uint16)
    v = rng.integers(0, 65536, size=(rows, hkv, d), dtype=np.uint16)
    acc = np.full((n_req, max_out), -7, dtype=np.int32)
    cnt = np.zeros(n_req, dtype=np.int32)
    for r in range(n_req):
        m = int(rng.integers(0, min(max_out - 1, ns[r]) + 1))
        lo = 1 if keep_root else 0                                     # with the root kept the list holds children only
        m = min(m, int(ns[r]) - lo)
        path = np.sort(lo + rng.choice(ns[r] - lo, size=m, replace=False)).astype(np.int32)
        if r == 1:
            path = np.arange(lo, lo + m, dtype=np.int32)              # already in place
        if r == 3:
            m, path = 0, np.zeros(0, np.int32)                         # only a drawn token
        if r == 4:
            m = -1                                                     # nothing emitted at all
        if r == 2 and ns[r] > 4:
            path = np.arange(1, min(ns[r], max_out - 1), dtype=np.int32)   # every move overlaps the previous one
            m = len(path)
        if m < 0:
            cnt[r] = 0
            continue
        acc[r, :m] = path
        acc[r, m] = -1                                                 # the drawn token
        cnt[r] = m + 1
    rk, rv = k.copy(), v.copy()
    want_L = np.zeros(n_req, np.int32)
    for r in range(n_req):
        want_L[r] = orc.compact_kv(rk, offs[r], Ls[r], acc[r, :cnt[r]], keep_root=keep_root)
        orc.compact_kv(rv, offs[r], Ls[r], acc[r, :cnt[r]], keep_root=keep_root)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    dk, dv = t(k.view(np.int16)), t(v.view(np.int16))
    newL = torch.zeros(n_req, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv(dk, dv, t(offs), t(Ls.astype(np.int32)), t(acc), t(cnt), n_req, max_out, hkv, d, newL,
                        keep_root=keep_root)
    torch.cuda.synchronize()
    assert np.array_equal(dk.cpu().numpy().view(np.uint16), rk)
    assert np.array_equal(dv.cpu().numpy().view(np.uint16), rv)
    assert np.array_equal(newL.cpu().numpy(), want_L)


def test_verify_then_compact_then_attend(B):
    """The three device steps in a row: verification picks a path, compaction moves its K/V rows, and
    a one-node attention over the new prefix matches the oracle over the gathered cache."""
    import torch
    from paper_2410_11744_b200 import runner as R
    rng = np.random.default_rng(21)
    parents = wl.greedy_tree(rng, 48, 6, 0.3)
    L = 200
    w = wl.make_custom(31, 8, 2, 128, [L], [parents])
    case = wl.make_verify_case(5, 4096, [parents], sharpness=3.0, disagreement=0.4)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    out_t = torch.zeros((1, 64), dtype=torch.int32, device=dev)
    out_n = torch.zeros((1, 64), dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_verify_tree(t(parents), t(case.tokens[0]), t(case.draft_probs), t(case.target_probs), t(case.accept_u),
                         t(case.sample_u), t(case.node_offsets), 1, 48, 4096, out_t, out_n, cnt, 64, bonus_at_leaf=True)
    batch = R.DeviceBatch(w)
    newL = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv(batch.k, batch.v, t(np.zeros(1, np.int64)), t(np.array([L], np.int32)), out_n, cnt, 1, 64, 2, 128, newL,
                        keep_root=True)
    torch.cuda.synchronize()
    listed = [int(a) for a in out_n[0, :int(cnt.item())].cpu().numpy()]
    path = [a for a in listed if a >= 0]
    assert 0 not in path                                                 # the kernel lists accepted children only
    k2, v2 = w.k.copy(), w.v.copy()
    want = orc.compact_kv(k2, 0, L, listed, keep_root=True)
    orc.compact_kv(v2, 0, L, listed, keep_root=True)
    assert int(newL.item()) == want == L + 1 + len(path)                 # old prefix + root + accepted path
    assert np.array_equal(R.bf16_tensor_to_bits(batch.k), k2) and np.array_equal(R.bf16_tensor_to_bits(batch.v), v2)
    # the next step: a one-node tree whose own row follows the new prefix sees prefix + root + path, i.e. what
    # the oracle computes over those rows gathered by hand from the ORIGINAL cache
    new_L = want
    rows = list(range(L)) + [L] + [L + a for a in path] + [L + 47]       # node 47's row stands in for the new token's
    k3, v3 = w.k[rows], w.v[rows]
    w1 = wl.make_custom(32, 8, 2, 128, [new_L], [np.array([-1], np.int32)])
    w1.q[:] = w.q[47:48]
    w1.k[:], w1.v[:] = k3, v3
    ref = orc.tree_attention(w1.q, k3, v3, new_L, [-1])
    b1 = R.DeviceBatch(w1)
    b1.k[:new_L].copy_(batch.k[:new_L])                                  # the compacted device cache itself
    b1.v[:new_L].copy_(batch.v[:new_L])
    b1.step()
    _, _, out_bits, st = b1.results()
    assert st == 0
    err = np.abs(orc.bf16_bits_to_f64(out_bits) - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
