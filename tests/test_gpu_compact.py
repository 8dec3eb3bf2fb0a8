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


@pytest.mark.parametrize("hkv,d", [(8, 128), (32, 128), (1, 64), (2, 8)])
def test_compact_matches_oracle(B, hkv, d):
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
        path = np.sort(rng.choice(ns[r], size=m, replace=False)).astype(np.int32)
        if r == 1:
            path = np.arange(m, dtype=np.int32)                       # already in place
        if r == 2 and ns[r] > 4:
            path = np.arange(1, min(ns[r], max_out - 1), dtype=np.int32)   # every move overlaps the previous one
            m = len(path)
        acc[r, :m] = path
        acc[r, m] = -1                                                 # the drawn token
        cnt[r] = m + 1
    rk, rv = k.copy(), v.copy()
    want_L = np.zeros(n_req, np.int32)
    for r in range(n_req):
        want_L[r] = orc.compact_kv(rk, offs[r], Ls[r], acc[r, :cnt[r]])
        orc.compact_kv(rv, offs[r], Ls[r], acc[r, :cnt[r]])
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    dk, dv = t(k.view(np.int16)), t(v.view(np.int16))
    newL = torch.zeros(n_req, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv(dk, dv, t(offs), t(Ls.astype(np.int32)), t(acc), t(cnt), n_req, max_out, hkv, d, newL)
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
    B.dyspec_compact_kv(batch.k, batch.v, t(np.zeros(1, np.int64)), t(np.array([L], np.int32)), out_n, cnt, 1, 64, 2, 128, newL)
    torch.cuda.synchronize()
    path = [int(a) for a in out_n[0, :int(cnt.item())].cpu().numpy() if a >= 0]
    k2, v2 = w.k.copy(), w.v.copy()
    want = orc.compact_kv(k2, 0, L, path)
    orc.compact_kv(v2, 0, L, path)
    assert int(newL.item()) == want == L + len(path)
    assert np.array_equal(R.bf16_tensor_to_bits(batch.k), k2) and np.array_equal(R.bf16_tensor_to_bits(batch.v), v2)
