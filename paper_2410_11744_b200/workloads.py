"""Seeded synthetic inputs for tree-verify attention.

This module only *draws inputs*: draft-tree topologies, prefix lengths and random
bf16 Q/K/V tensors shaped like the Llama2-7B / Llama2-70B attention layers the
paper evaluates (Sec. 5.1; App. C.1 uses 64 heads x head_dim 128).  It holds
none of the method's arithmetic (no masks, no attention) and is used by the
tests, the benchmark and the oracle-side scripts alike.  It imports neither the
CUDA binding nor the oracle.

Tree recipe: a deterministic-score form of the paper's greedy expansion
(Sec. 4.1-4.2, Algorithm 1; weight model of App. D): node 0 is the root (parent
-1, score 1).  When a node is created it draws p ~ Dirichlet(alpha * 1_c) and
pushes its c candidate children with score(node) * p_j on a max-heap; the best
candidate is popped and becomes the next node, so parent[i] < i, until n nodes
exist.  Ties: higher score first, then earlier push.

bf16 values are carried as uint16 bit patterns (numpy has no bf16 type).
"""
from __future__ import annotations

import heapq
import math
from dataclasses import dataclass, field
from typing import List

import numpy as np

MASTER_SEED = 241011744


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns.

    Input generation only: the values fed to both implementations are these bits.
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)   # finite inputs: no uint32 overflow below
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def greedy_tree(rng: np.random.Generator, n_nodes: int, n_candidates: int, alpha: float) -> np.ndarray:
    """Parent array (int32, parents[0] = -1, parents[i] < i) of a greedy best-first tree."""
    parents = np.full(n_nodes, -1, dtype=np.int32)
    if n_nodes == 0:
        return parents
    heap: list = []
    push_id = 0

    def expand(node: int, log_score: float) -> None:
        nonlocal push_id
        p = rng.dirichlet(np.full(n_candidates, alpha, dtype=np.float64))
        for j in range(n_candidates):
            lp = math.log(p[j]) if p[j] > 0.0 else -math.inf
            heapq.heappush(heap, (-(log_score + lp), push_id, node))
            push_id += 1

    expand(0, 0.0)
    for i in range(1, n_nodes):
        neg_log_score, _, parent = heapq.heappop(heap)
        parents[i] = parent
        expand(i, -neg_log_score)
    return parents


def chain_tree(n_nodes: int) -> np.ndarray:
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def star_forest(n_nodes: int) -> np.ndarray:
    """Every node is its own root (parent -1)."""
    return np.full(n_nodes, -1, dtype=np.int32)


def random_tree(rng: np.random.Generator, n_nodes: int, p_root: float = 0.0) -> np.ndarray:
    """Uniform random recursive tree / forest with parents[i] < i."""
    parents = np.full(n_nodes, -1, dtype=np.int32)
    for i in range(1, n_nodes):
        if rng.random() >= p_root:
            parents[i] = int(rng.integers(0, i))
    return parents


@dataclass
class Workload:
    """One ragged batch of verification requests (all arrays host-side numpy)."""
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prefix_len: np.ndarray          # int32 [n_req]
    n_nodes: np.ndarray             # int32 [n_req]
    parents: List[np.ndarray]       # per request int32 [n_nodes[r]], request-local indices
    q: np.ndarray                   # uint16 bf16 bits [sum n_nodes][H_q][D]
    k: np.ndarray                   # uint16 bf16 bits [total_rows][H_kv][D]
    v: np.ndarray                   # same layout as k
    kv_row_offset: np.ndarray       # int64 [n_req]: row of request r's token 0 in k / v
    meta: dict = field(default_factory=dict)

    @property
    def n_req(self) -> int:
        return int(self.prefix_len.shape[0])

    @property
    def node_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.n_nodes)]).astype(np.int32)

    @property
    def parents_concat(self) -> np.ndarray:
        if len(self.parents) == 0:
            return np.zeros(0, dtype=np.int32)
        return np.concatenate(self.parents).astype(np.int32)

    @property
    def total_nodes(self) -> int:
        return int(self.n_nodes.sum())

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    def request(self, r: int):
        """(q, k, v, parents, prefix_len) slices of request r; k/v hold prefix rows then tree rows."""
        no = self.node_offsets
        o = int(self.kv_row_offset[r])
        rows = int(self.prefix_len[r]) + int(self.n_nodes[r])
        return (self.q[no[r]:no[r + 1]], self.k[o:o + rows], self.v[o:o + rows],
                self.parents[r], int(self.prefix_len[r]))


def _normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(size=shape, dtype=np.float32))


def assemble(name, rng, n_q_heads, n_kv_heads, head_dim, prefix_len, parents_list, meta=None) -> Workload:
    """Draw Q, K, V ~ N(0,1) (in that order) for given trees and prefix lengths, requests packed back to back."""
    prefix_len = np.asarray(prefix_len, dtype=np.int32)
    n_nodes = np.asarray([len(p) for p in parents_list], dtype=np.int32)
    rows = prefix_len.astype(np.int64) + n_nodes.astype(np.int64)
    kv_off = np.concatenate([[0], np.cumsum(rows)[:-1]]).astype(np.int64) if len(rows) else np.zeros(0, np.int64)
    total_rows = int(rows.sum())
    total_nodes = int(n_nodes.sum())
    q = _normal_bf16(rng, (total_nodes, n_q_heads, head_dim))
    k = _normal_bf16(rng, (total_rows, n_kv_heads, head_dim))
    v = _normal_bf16(rng, (total_rows, n_kv_heads, head_dim))
    return Workload(name, n_q_heads, n_kv_heads, head_dim, prefix_len, n_nodes,
                    [np.asarray(p, dtype=np.int32) for p in parents_list], q, k, v, kv_off, meta or {})


# Shapes of the five benchmark configurations: (H_q, H_kv, D, prefix_len, n_nodes, candidates, alpha).
_FIXED = {
    1: dict(name="c1_tiny_4x4_d64_L128_n16", hq=4, hkv=4, d=64, L=128, n=16, c=4, alpha=0.3),
    2: dict(name="c2_llama2_7b_L1024_n64", hq=32, hkv=32, d=128, L=1024, n=64, c=8, alpha=0.3),
    3: dict(name="c3_llama2_7b_L4096_n256", hq=32, hkv=32, d=128, L=4096, n=256, c=8, alpha=0.1),
    4: dict(name="c4_llama2_70b_L2048_n512", hq=64, hkv=8, d=128, L=2048, n=512, c=8, alpha=0.3),
}


def make_config(index: int, seed: int | None = None) -> Workload:
    """Config `index` in 1..5 (1 = tiny ... 5 = ragged batch of 8 Llama2-70B-shaped requests)."""
    if seed is None:
        seed = MASTER_SEED + index
    rng = np.random.default_rng(seed)
    if index in _FIXED:
        c = _FIXED[index]
        parents = greedy_tree(rng, c["n"], c["c"], c["alpha"])
        return assemble(c["name"], rng, c["hq"], c["hkv"], c["d"], [c["L"]], [parents],
                        dict(config=index, seed=seed, candidates=c["c"], alpha=[c["alpha"]]))
    if index == 5:
        n_req = 8
        Ls, ns, alphas, trees = [], [], [], []
        for _ in range(n_req):
            L = int(round(math.exp(rng.uniform(math.log(512.0), math.log(8192.0)))))
            n = int(rng.integers(32, 769))
            a = float(rng.uniform(0.05, 1.0))
            Ls.append(L); ns.append(n); alphas.append(a)
            trees.append(greedy_tree(rng, n, 8, a))
        return assemble("c5_ragged8_llama2_70b", rng, 64, 8, 128, Ls, trees,
                        dict(config=5, seed=seed, candidates=8, alpha=alphas))
    raise ValueError(f"config index must be 1..5, got {index}")


def make_custom(seed: int, n_q_heads: int, n_kv_heads: int, head_dim: int, prefix_len, parents_list,
                name: str = "custom") -> Workload:
    return assemble(name, np.random.default_rng(seed), n_q_heads, n_kv_heads, head_dim, prefix_len, parents_list,
                    dict(seed=seed))


def make_random_tree_case(n_nodes: int, seed: int | None = None, n_heads: int = 64, head_dim: int = 128,
                          prefix_len: int = 0) -> Workload:
    """The random-tree attention experiment of App. C.1 (Table 5): one request, 64 heads of dimension
    128, no prefix, a uniform random recursive tree of n_nodes tokens in creation order."""
    if seed is None:
        seed = MASTER_SEED + 5000 + n_nodes
    rng = np.random.default_rng(seed)
    parents = random_tree(rng, n_nodes)
    return assemble(f"random_tree_n{n_nodes}_h{n_heads}_d{head_dim}_L{prefix_len}", rng, n_heads, n_heads, head_dim,
                    [prefix_len], [parents], dict(seed=seed, experiment="random_tree"))


def permute_tree_tokens(w: Workload, orders: List[np.ndarray], new_parents: List[np.ndarray]) -> Workload:
    """The same requests with their tree tokens renumbered: new token k of request r is old token
    orders[r][k] (its Q row and its K/V row move with it); new_parents[r] is the parent array in the
    new numbering (computed by whoever chose the order; this function only moves rows)."""
    q, k, v = w.q.copy(), w.k.copy(), w.v.copy()
    no = w.node_offsets
    for r in range(w.n_req):
        order = np.asarray(orders[r], dtype=np.int64)
        base = int(w.kv_row_offset[r]) + int(w.prefix_len[r])
        q[no[r]:no[r + 1]] = w.q[no[r] + order]
        k[base:base + len(order)] = w.k[base + order]
        v[base:base + len(order)] = w.v[base + order]
    return Workload(w.name + "_reordered", w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len.copy(), w.n_nodes.copy(),
                    [np.asarray(p, dtype=np.int32) for p in new_parents], q, k, v, w.kv_row_offset.copy(),
                    dict(w.meta, reordered=True))


@dataclass
class VerifyCase:
    """Inputs of the tree verification (Algorithm 3) for a ragged batch: all arrays host-side numpy."""
    name: str
    vocab: int
    node_offsets: np.ndarray        # int32 [n_req + 1]
    parents: List[np.ndarray]       # per request int32 [n]
    tokens: List[np.ndarray]        # per request int32 [n]: token carried by each node (root: 0)
    draft_probs: np.ndarray         # float32 [N][vocab]
    target_probs: np.ndarray        # float32 [N][vocab]
    accept_u: np.ndarray            # float32 [N]
    sample_u: np.ndarray            # float32 [N]


def _softmax_rows(x: np.ndarray) -> np.ndarray:
    x = x - x.max(axis=1, keepdims=True)
    e = np.exp(x)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def make_verify_case(seed: int, vocab: int, parents_list, sharpness: float = 4.0, disagreement: float = 1.0,
                     same: bool = False, name: str = "verify") -> VerifyCase:
    """Draft rows = softmax(sharpness * N(0,1) logits); target rows = softmax of the same logits plus
    disagreement * N(0,1) noise (same=True: identical rows).  The children of a node carry tokens drawn
    from the node's draft row without replacement, in child order, which is how a draft tree comes
    about (Sec. 4.1); when the row runs out of mass the remaining children get unused tokens."""
    rng = np.random.default_rng(seed)
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents_list])]).astype(np.int32)
    N = int(offs[-1])
    logits = rng.standard_normal((N, vocab)).astype(np.float32) * np.float32(sharpness)
    draft = _softmax_rows(logits)
    target = draft.copy() if same else _softmax_rows(logits + np.float32(disagreement) * rng.standard_normal((N, vocab)).astype(np.float32))
    tokens = []
    for r, parents in enumerate(parents_list):
        n = len(parents)
        tok = np.zeros(n, dtype=np.int32)
        children = [[] for _ in range(n)]
        for i in range(1, n):
            if parents[i] >= 0:
                children[int(parents[i])].append(i)
        for u in range(n):
            if not children[u]:
                continue
            d = draft[offs[r] + u].astype(np.float64).copy()
            for c in children[u]:
                if d.sum() > 0:
                    y = int(rng.choice(vocab, p=d / d.sum()))
                else:
                    y = int(np.flatnonzero(draft[offs[r] + u] == 0)[0]) if (draft[offs[r] + u] == 0).any() else 0
                tok[c] = y
                d[y] = 0.0
        tokens.append(tok)
    return VerifyCase(name, vocab, offs, [np.asarray(p, np.int32) for p in parents_list], tokens, draft, target,
                      rng.random(N, dtype=np.float32), rng.random(N, dtype=np.float32))


def make_draft_table(seed: int, n_rows: int, vocab: int, sharpness: float = 3.0, n_uniforms: int = 4099,
                     zipf: bool = False):
    """The table-lookup draft model of the tree-construction kernels: n_rows distributions over the
    vocabulary and a table of U(0,1) numbers.  Rows are softmax(sharpness * N(0,1) logits), or with
    zipf=True language-model-like: p ~ rank^-a with a ~ U(1.1, 2.2) per row over a random permutation
    of the tokens (top token 0.2 - 0.7), fp32."""
    rng = np.random.default_rng(seed)
    if zipf:
        rows = np.empty((n_rows, vocab), dtype=np.float32)
        ranks = np.arange(1, vocab + 1, dtype=np.float64)
        for i in range(n_rows):
            p = ranks ** (-rng.uniform(1.1, 2.2))
            rows[i, rng.permutation(vocab)] = (p / p.sum()).astype(np.float32)
    else:
        rows = _softmax_rows(rng.standard_normal((n_rows, vocab)).astype(np.float32) * np.float32(sharpness))
    return rows, rng.random(n_uniforms, dtype=np.float32)


@dataclass
class PagedWorkload:
    """A Workload whose KV cache is a pool of pages: prefix token t of request r lies at pool row
    page_table[r, t // page_size] * page_size + t % page_size; the tree rows of request r are the
    contiguous pool rows tree_row_offset[r] .. + n_nodes[r]."""
    base: Workload                  # q, parents, prefix_len, n_nodes as in the contiguous layout
    page_size: int
    page_table: np.ndarray          # int32 [n_req][pages_per_req], -1 = no page
    tree_row_offset: np.ndarray     # int64 [n_req]
    k: np.ndarray                   # uint16 bf16 bits [pool_rows][H_kv][D]
    v: np.ndarray

    @property
    def pages_per_req(self) -> int:
        return int(self.page_table.shape[1])

    @property
    def pool_rows(self) -> int:
        return int(self.k.shape[0])


def to_paged(w: Workload, page_size: int, seed: int = 0, room_for_accepted: bool = True,
             tree_in_pages: bool = False) -> PagedWorkload:
    """Scatters w's contiguous cache into a paged pool.  Every request gets enough pages for its prefix
    (plus its tree size when room_for_accepted, so that accepted tokens have somewhere to go), the page
    numbers of all requests are shuffled together, rows of a page past the prefix hold finite filler
    (large values, so that a key that leaks through a mask shows), and the tree rows follow the pages
    with odd gaps between requests.  With tree_in_pages the tree rows are tokens L .. L + n - 1 of the
    paged sequence instead (tree_row_offset is then None)."""
    rng = np.random.default_rng(seed + 99173)
    n_req = w.n_req
    room_for_accepted = room_for_accepted or tree_in_pages
    need = [-(-(int(w.prefix_len[r]) + (int(w.n_nodes[r]) if room_for_accepted else 0)) // page_size) for r in range(n_req)]
    pages_per_req = max(need + [1])
    n_pages = sum(need) + 2                                   # two pages nobody owns
    ids = rng.permutation(n_pages)
    page_table = np.full((n_req, pages_per_req), -1, dtype=np.int32)
    at = 0
    for r in range(n_req):
        page_table[r, :need[r]] = ids[at:at + need[r]]
        at += need[r]
    tree_row_offset = np.zeros(n_req, dtype=np.int64)
    row = n_pages * page_size
    for r in range(n_req):
        row += 3 + 2 * r
        tree_row_offset[r] = row
        row += int(w.n_nodes[r])
    pool_rows = row + 5
    shape = (pool_rows,) + tuple(w.k.shape[1:])
    filler = np.array([0x4248, 0xC248, 0x4170, 0xC170], dtype=np.uint16)     # bf16 50, -50, 15, -15
    k = filler[rng.integers(0, 4, size=shape)]
    v = filler[rng.integers(0, 4, size=shape)]
    for r in range(n_req):
        o, L, n = int(w.kv_row_offset[r]), int(w.prefix_len[r]), int(w.n_nodes[r])
        for t0 in range(0, L, page_size):
            cnt = min(page_size, L - t0)
            dst = int(page_table[r, t0 // page_size]) * page_size
            k[dst:dst + cnt] = w.k[o + t0:o + t0 + cnt]
            v[dst:dst + cnt] = w.v[o + t0:o + t0 + cnt]
        if tree_in_pages:
            for t in range(L, L + n):
                dst = int(page_table[r, t // page_size]) * page_size + t % page_size
                k[dst] = w.k[o + t]
                v[dst] = w.v[o + t]
            continue
        t = int(tree_row_offset[r])
        k[t:t + n] = w.k[o + L:o + L + n]
        v[t:t + n] = w.v[o + L:o + L + n]
    return PagedWorkload(w, int(page_size), page_table, None if tree_in_pages else tree_row_offset, k, v)
