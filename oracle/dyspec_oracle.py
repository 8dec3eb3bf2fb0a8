"""fp64 CPU oracle for tree-verify attention.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this file; the product (the CUDA library and its binding) never does, and this
file imports nothing from the product.  It is deliberately plain and slow.

What it computes (every function names the passage of the paper it follows):

* The tree attention mask of Sec. 2 ("Tree Attention", the mask(A) equation): a
  query node may see key node j exactly when j is one of its ancestors.  As in
  ordinary causal attention (same paragraph) a token also sees itself, so the
  visible set of node i is A(i) = {i} + ancestors(i).
* Parallel verification (Sec. 2, "Speculative Decoding"; App. C: the prompt is
  part of the attention mask): every tree token is scored by the target model
  as if its root-to-node path had been decoded after the prefix, i.e. node i
  attends to all prefix rows and to the tree rows in A(i):

      s_t = scale * <q[i,h,:], k[t,h_kv,:]>,  p = softmax_t over visible t,
      o[i,h,:] = sum_t p_t * v[t,h_kv,:],     h_kv = h // (H_q / H_kv).

  The method reaches exactly this result (it is not an approximation), so the
  oracle is this definition written out with a dense boolean mask, in fp64.

Parity status: every function below is pinned by tests/test_oracle_pins.py
(chain == library causal attention, star == prefix+self, brute force per path
in pure Python, closed forms, hand-written mask fixture, relabelling
invariance; visible_pair_count by the chain, star and binary-tree closed forms
and a pair-by-pair count); the token-reorder functions at the end (App. C) are pinned by
tests/test_reorder_pins.py (the block counts the paper prints in Table 5,
closed forms, a hand example, subtree contiguity, attention invariance);
verify_tree (Algorithm 3) by tests/test_verify_pins.py (the output distribution
equals the target's, Draft == Target accepts every first branch, closed-form
acceptance rates, forced rejections, the all-zero early exit); the tree
construction (Algorithms 1 and 2) by tests/test_construct_pins.py (values
decrease, the closed form of the estimated acceptance rate in raw draft
probabilities, Algorithm 2 at the last value == Algorithm 1, guesses at a
position are draws without replacement); compact_kv by
tests/test_compact_pins.py (hand example, no-op on a chain prefix, attention
over the compacted cache == attention along the accepted path); the paged
forms by tests/test_paged_pins.py (a hand-written page table, the identity
table == the contiguous layout, any scattering of the pages leaves the
attention bit-identical, compaction == the contiguous one read back through
the table).
Nothing here is "parity unpinned".

Readings where the paper is silent: scale = 1/sqrt(head_dim); consecutive query
heads share a KV head; tree K/V rows follow the prefix rows in node order;
masks are packed LSB-first in uint32 words; the DFS renumbering visits roots
and children in increasing index (the order that reproduces Table 5);
Algorithm 3 draws its acceptance number from U(0,1) (printed as N(0,1)), the
branches of a node are its children in increasing index, and the final token
is drawn from the residual by inverse CDF in token order; Algorithm 1 samples
the token before it adds the node, Algorithm 2 expands while v >= t, the draft
model is a table lookup keyed by tree position (see build_tree_greedy); in
the paged layout the tree rows are a contiguous run outside the prefix pages.
"""
from __future__ import annotations

import math
from typing import List, Sequence

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening: a bf16 value is the top 16 bits of an IEEE fp32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def check_parents(parents: Sequence[int]) -> None:
    """A valid parent array has parents[i] == -1 (a root) or 0 <= parents[i] < i."""
    for i, p in enumerate(parents):
        p = int(p)
        if p < -1 or p >= i:
            raise ValueError(f"parents[{i}] = {p} is not in {{-1}} U [0, {i})")


def visible_nodes(parents: Sequence[int], i: int) -> List[int]:
    """A(i): node i followed by its ancestors, found by walking the parent links (Sec. 2, mask(A))."""
    out = []
    j = int(i)
    while j != -1:
        out.append(j)
        j = int(parents[j])
    return out


def tree_mask_matrix(parents: Sequence[int]) -> np.ndarray:
    """Boolean [n][n]; entry [i][j] is True iff query node i may attend to key node j (j in A(i))."""
    check_parents(parents)
    n = len(parents)
    m = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in visible_nodes(parents, i):
            m[i, j] = True
    return m


def build_tree_mask(parents: Sequence[int], words_per_row: int):
    """Packed ancestor bitmasks and depths.

    bits[i][w] has bit b (LSB = bit 0) set iff node 32*w + b is in A(i); unused bits are 0.
    depth[i] = number of ancestors of i (roots have depth 0).
    """
    check_parents(parents)
    n = len(parents)
    if 32 * words_per_row < n:
        raise ValueError("words_per_row too small")
    bits = np.zeros((n, words_per_row), dtype=np.uint32)
    depths = np.zeros(n, dtype=np.int32)
    for i in range(n):
        vis = visible_nodes(parents, i)
        for j in vis:
            bits[i, j // 32] |= np.uint32(1 << (j % 32))
        depths[i] = len(vis) - 1
    return bits, depths


def tree_attention(q_bits, k_bits, v_bits, prefix_len: int, parents: Sequence[int], scale: float | None = None):
    """Tree-verify attention for one request, fp64.

    q_bits [n][H_q][D], k_bits / v_bits [prefix_len + n][H_kv][D] (bf16 bit patterns; tree row j
    sits at row prefix_len + j).  Returns float64 [n][H_q][D].
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    n, hq, d = q.shape
    rows, hkv, dk = k.shape
    L = int(prefix_len)
    if rows != L + n or dk != d or v.shape != k.shape or hq % hkv != 0 or len(parents) != n:
        raise ValueError("inconsistent shapes")
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(d)
    g = hq // hkv
    allowed = np.ones((n, L + n), dtype=bool)           # prefix: always visible
    allowed[:, L:] = tree_mask_matrix(parents)          # tree block: ancestors and self
    out = np.zeros((n, hq, d), dtype=np.float64)
    for h in range(hq):
        kh = k[:, h // g, :]
        vh = v[:, h // g, :]
        s = scale * (q[:, h, :] @ kh.T)                 # [n][L+n]
        s = np.where(allowed, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ vh
    return out


def tree_attention_nodes(q_bits, k_bits, v_bits, prefix_len: int, parents: Sequence[int], nodes: Sequence[int],
                         scale: float | None = None):
    """The same definition evaluated only for the query nodes listed in `nodes` -> float64 [len(nodes)][H_q][D].

    Used to check sampled outputs at sizes where all rows would take too long.
    """
    check_parents(parents)
    L = int(prefix_len)
    nodes = [int(i) for i in nodes]
    q = bf16_bits_to_f64(np.asarray(q_bits)[nodes])
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    m, hq, d = q.shape
    hkv = k.shape[1]
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(d)
    g = hq // hkv
    out = np.zeros((m, hq, d), dtype=np.float64)
    for a, i in enumerate(nodes):
        rows = list(range(L)) + [L + j for j in sorted(visible_nodes(parents, i))]
        for h in range(hq):
            kh = k[rows, h // g, :]
            vh = v[rows, h // g, :]
            s = scale * (kh @ q[a, h, :])
            p = np.exp(s - s.max())
            out[a, h, :] = (p / p.sum()) @ vh
    return out


def tree_attention_ragged(q_bits, k_bits, v_bits, prefix_len, n_nodes, kv_row_offset, parents_list,
                          scale: float | None = None):
    """Ragged batch: requests are independent; request r owns q rows node_offsets[r]..., kv rows
    kv_row_offset[r] .. + prefix_len[r] + n_nodes[r].  Returns float64 [sum n][H_q][D]."""
    outs = []
    qo = 0
    for r in range(len(prefix_len)):
        n = int(n_nodes[r])
        o = int(kv_row_offset[r])
        rows = int(prefix_len[r]) + n
        if n:
            outs.append(tree_attention(q_bits[qo:qo + n], k_bits[o:o + rows], v_bits[o:o + rows],
                                       int(prefix_len[r]), parents_list[r], scale))
        qo += n
    if not outs:
        return np.zeros((0,) + tuple(q_bits.shape[1:]), dtype=np.float64)
    return np.concatenate(outs, axis=0)


def build_tree_mask_ragged(parents_list, words_per_row: int):
    """Masks and depths of every request, rows concatenated in request order."""
    bits, depths = [], []
    for p in parents_list:
        b, dpt = build_tree_mask(p, words_per_row)
        bits.append(b)
        depths.append(dpt)
    if not bits:
        return np.zeros((0, words_per_row), np.uint32), np.zeros(0, np.int32)
    return np.concatenate(bits, axis=0), np.concatenate(depths)


def visible_pair_count(prefix_len, parents_list) -> int:
    """Sum over nodes of (prefix_len + depth + 1): the number of (query, key) pairs the definition uses."""
    total = 0
    for L, p in zip(prefix_len, parents_list):
        for i in range(len(p)):
            total += int(L) + len(visible_nodes(p, i))
    return total


# ----------------------------------------------------------------------------------------------------
# Block-sparsity friendly token order (App. C): depth-first renumbering and the non-zero block count.
# ----------------------------------------------------------------------------------------------------
def dfs_order(parents: Sequence[int]) -> List[int]:
    """Depth-first (pre-order) visiting sequence of the forest: order[k] = old index of the node that
    gets new index k.  Roots, and the children of a node, are visited in increasing old index (App. C:
    DySpec renumbers nodes in DFS order because it approximates heavy-path order)."""
    check_parents(parents)
    n = len(parents)
    children: List[List[int]] = [[] for _ in range(n)]
    roots: List[int] = []
    for i in range(n):
        p = int(parents[i])
        if p < 0:
            roots.append(i)
        else:
            children[p].append(i)
    order: List[int] = []

    def visit(u: int) -> None:
        order.append(u)
        for c in children[u]:
            visit(c)

    import sys
    limit = sys.getrecursionlimit()
    sys.setrecursionlimit(max(limit, n + 100))
    try:
        for r in roots:
            visit(r)
    finally:
        sys.setrecursionlimit(limit)
    return order


def relabel_tree(parents: Sequence[int], order: Sequence[int]):
    """Parent array after renumbering: new node k is old node order[k].  Returns (new_parents int32 [n],
    new_of_old int32 [n]).  For a DFS order the result again satisfies new_parents[k] < k."""
    n = len(parents)
    new_of_old = np.full(n, -1, dtype=np.int32)
    for k, old in enumerate(order):
        new_of_old[int(old)] = k
    new_parents = np.full(n, -1, dtype=np.int32)
    for k, old in enumerate(order):
        p = int(parents[int(old)])
        new_parents[k] = -1 if p < 0 else int(new_of_old[p])
    return new_parents, new_of_old


def mask_block_count(parents: Sequence[int], block: int = 32) -> int:
    """Number of block x block tiles of the tree attention mask (ancestors and self) that hold at
    least one visible entry: the workload measure of App. C.1, Table 5."""
    m = tree_mask_matrix(parents)
    n = m.shape[0]
    t = (n + block - 1) // block
    count = 0
    for a in range(t):
        for b in range(t):
            if m[a * block:(a + 1) * block, b * block:(b + 1) * block].any():
                count += 1
    return count


# ----------------------------------------------------------------------------------------------------
# Verification of the token tree against the target model (App. "Verification", Algorithm 3).
# ----------------------------------------------------------------------------------------------------
def verify_tree(parents: Sequence[int], tokens: Sequence[int], draft_probs, target_probs, accept_u, sample_u,
                bonus_at_leaf: bool = False):
    """Algorithm 3 (multi-branch rejection sampling along the tree), in fp64.

    parents[i], tokens[i]  the tree and the token each node carries (the root's token is not used);
                           the branches of a node are its children in increasing index
    draft_probs[i][v]      Draft(node i, v): the distribution node i's children were drawn from
    target_probs[i][v]     Target(node i, v)
    accept_u[i]            the number drawn when child i is tried; the paper prints c ~ N(0,1), which
                           cannot be meant for an accept-with-probability-R[y]/D[y] test: read U(0,1)
    sample_u[i]            the U(0,1) number used if the walk ends at node i and a token is drawn from
                           the residual R there (inverse CDF: the first v with cumsum(R)[v] > u * sum(R))
    Roots other than node 0 are ignored (the walk starts at node 0).  As printed, the loop runs while
    the current node has branches, so a walk that reaches a leaf ends there without a further token;
    bonus_at_leaf=True adds the usual extra token drawn from Target(leaf, .) instead.

    Returns (accepted_tokens, accepted_nodes, margins): the token sequence A, the nodes that were
    accepted (the final, sampled token has no node), and for every decision taken a pair (kind,
    distance of the deciding number from its threshold): ("accept", |c - R[y]/D[y]|) or ("sample",
    distance of u from the nearer edge of the drawn token's CDF interval), so that a lower-precision
    implementation can be excused where the decision was a coin toss.
    """
    check_parents(parents)
    n = len(parents)
    D_all = np.asarray(draft_probs, dtype=np.float64)
    T_all = np.asarray(target_probs, dtype=np.float64)
    children: List[List[int]] = [[] for _ in range(n)]
    for i in range(1, n):
        if int(parents[i]) >= 0:
            children[int(parents[i])].append(i)
    accepted_tokens: List[int] = []
    accepted_nodes: List[int] = []
    margins: List[tuple] = []
    if n == 0:
        return accepted_tokens, accepted_nodes, margins
    cur = 0
    while True:
        if not children[cur] and not bonus_at_leaf:
            break
        R = T_all[cur].copy()
        moved = False
        if children[cur]:
            D = D_all[cur].copy()
            for child in children[cur]:
                y = int(tokens[child])
                c = float(accept_u[child])
                ratio = R[y] / D[y] if D[y] > 0 else (np.inf if R[y] > 0 else 0.0)
                margins.append(("accept", abs(c - ratio)))
                if c <= ratio:
                    accepted_tokens.append(y)
                    accepted_nodes.append(child)
                    cur = child
                    moved = True
                    break
                R = np.maximum(R - D, 0.0)
                if R.sum() > 0:
                    R = R / R.sum()
                D[y] = 0.0
                if not (D > 0).any():
                    break
                D = D / D.sum()
        if not moved:
            total = R.sum()
            if total <= 0:              # nothing left to sample from (cannot happen when Draft != Target on the support)
                R = T_all[cur].copy()
                total = R.sum()
            cdf = np.cumsum(R)
            target = float(sample_u[cur]) * total
            y = int(np.searchsorted(cdf, target, side="right"))
            y = min(y, len(R) - 1)
            lo = cdf[y - 1] if y > 0 else 0.0
            margins.append(("sample", min(abs(target - lo), abs(cdf[y] - target)) / total))
            accepted_tokens.append(y)
            break
    return accepted_tokens, accepted_nodes, margins


# ----------------------------------------------------------------------------------------------------
# Construction of the draft token tree (Sec. 4.1-4.3, Algorithm 1; App. B, Algorithm 2).
#
# The draft model is abstracted as a table: the distribution that follows a tree position is a row of
# `rows`, chosen by a fixed integer function of the position (row of the parent, token), and the
# uniform number used by the j-th sampling at a position is an entry of `uniforms` chosen the same way.
# Both algorithms therefore see the same distribution and draw the same token for the same (position,
# attempt), which is what makes the paper's statement "with the threshold set to the value of the last
# node, Algorithm 2 gives exactly the tree of Algorithm 1" checkable.
# ----------------------------------------------------------------------------------------------------
def draft_row_of_child(parent_row: int, token: int, n_rows: int) -> int:
    return ((parent_row * 2654435761 + (token + 1) * 40503) % (1 << 32)) % n_rows


def draft_uniform_index(row: int, attempt: int, n_uniforms: int) -> int:
    return ((row * 7919 + attempt * 104729 + 17) % (1 << 32)) % n_uniforms


def _sample_residual(raw_row: np.ndarray, taken: List[int], u: float):
    """Draws from norm(raw_row with the `taken` tokens zeroed) by inverse CDF in token order.
    Returns (token, its probability under that residual, margin of u from the CDF interval's edges)."""
    res = raw_row.astype(np.float64).copy()
    res[taken] = 0.0
    total = res.sum()
    cdf = np.cumsum(res)
    target = float(u) * total
    y = int(np.searchsorted(cdf, target, side="right"))
    y = min(y, len(res) - 1)
    lo = cdf[y - 1] if y > 0 else 0.0
    margin = min(abs(target - lo), abs(cdf[y] - target)) / total if total > 0 else 0.0
    return y, (res[y] / total if total > 0 else 0.0), margin


def build_tree_greedy(rows, uniforms, m: int, root_row: int = 0):
    """Algorithm 1: the tree of the m guesses with the largest estimated acceptance rate.

    A slot (v, position, attempt) stands for "the next sampling at this position"; the slot with the
    largest v is taken (ties: the one pushed first), a token is sampled from the position's residual
    distribution (the printed listing adds the node one line before it samples the token: read in the
    order that makes sense), the node is created, and two slots are pushed: the next sampling at the
    same position with v (1 - R[y]) and the first sampling under the new node with v R[y].

    Returns dict(parents, tokens, values, child_values, rows, margins): node 0 is the root (the last
    prompt token; value 1); values[k] is the slot value node k was created from, child_values[k] the
    value of the first sampling under it; margins as in verify_tree, plus ("order", gap between the
    best and the second best slot value, relative)."""
    rows = np.asarray(rows)
    T, Tu = rows.shape[0], len(uniforms)
    parents, tokens, values, child_values, node_rows = [-1], [0], [1.0], [1.0], [int(root_row) % rows.shape[0]]
    taken: List[List[int]] = [[]]
    slots = [(1.0, 0, 0)]                      # (v, position, attempt), in push order
    margins: List[tuple] = []
    while len(parents) - 1 < m and slots:
        best = max(range(len(slots)), key=lambda i: (slots[i][0], -i))
        if len(slots) > 1:
            second = max(s[0] for i, s in enumerate(slots) if i != best)
            margins.append(("order", (slots[best][0] - second) / max(slots[best][0], 1e-300)))
        v, pos, attempt = slots.pop(best)
        u = uniforms[draft_uniform_index(node_rows[pos], attempt, Tu)]
        y, r, mg = _sample_residual(rows[node_rows[pos]], taken[pos], u)
        margins.append(("sample", mg))
        k = len(parents)
        parents.append(pos); tokens.append(y); values.append(v); child_values.append(v * r)
        node_rows.append(draft_row_of_child(node_rows[pos], y, T))
        taken.append([])
        taken[pos].append(y)
        if 1.0 - r > 0.0:
            slots.append((v * (1.0 - r), pos, attempt + 1))
        slots.append((v * r, k, 0))
    return dict(parents=np.asarray(parents, np.int32), tokens=np.asarray(tokens, np.int32),
                values=np.asarray(values), child_values=np.asarray(child_values),
                rows=np.asarray(node_rows, np.int32), margins=margins)


def build_tree_threshold(rows, uniforms, threshold: float, max_nodes: int, root_row: int = 0):
    """Algorithm 2: layer by layer, every position keeps sampling while its estimated acceptance rate
    is at least `threshold` (the printed loop condition `v < t` would expand exactly the guesses the
    text says to drop: read `v >= t`).  Stops early when max_nodes guesses exist.  Same return value as
    build_tree_greedy (node order: by layer, then by parent, then by sampling order)."""
    rows = np.asarray(rows)
    T, Tu = rows.shape[0], len(uniforms)
    parents, tokens, values, child_values, node_rows = [-1], [0], [1.0], [1.0], [int(root_row) % rows.shape[0]]
    margins: List[tuple] = []
    leaves = [0]
    while leaves and len(parents) - 1 < max_nodes:
        new_leaves = []
        for node in leaves:
            v = child_values[node]
            taken: List[int] = []
            attempt = 0
            while v >= threshold and len(parents) - 1 < max_nodes:
                margins.append(("threshold", abs(v - threshold) / max(threshold, 1e-300)))
                u = uniforms[draft_uniform_index(node_rows[node], attempt, Tu)]
                y, r, mg = _sample_residual(rows[node_rows[node]], taken, u)
                margins.append(("sample", mg))
                k = len(parents)
                parents.append(node); tokens.append(y); values.append(v); child_values.append(v * r)
                node_rows.append(draft_row_of_child(node_rows[node], y, T))
                new_leaves.append(k)
                taken.append(y)
                v = v * (1.0 - r)
                attempt += 1
                if not (1.0 - r > 0.0):
                    break
            if v < threshold:
                margins.append(("threshold", abs(v - threshold) / max(threshold, 1e-300)))
        leaves = new_leaves
    return dict(parents=np.asarray(parents, np.int32), tokens=np.asarray(tokens, np.int32),
                values=np.asarray(values), child_values=np.asarray(child_values),
                rows=np.asarray(node_rows, np.int32), margins=margins)


# ----------------------------------------------------------------------------------------------------
# Keeping the accepted path in the KV cache (the step after verification; the paper only says that the
# accepted tokens extend the prefix, Sec. 2 / Algorithm 3).
# ----------------------------------------------------------------------------------------------------
def kept_nodes(accepted_nodes: Sequence[int], keep_root: bool) -> List[int]:
    """The tree nodes whose K/V rows survive a verification step, in sequence order.  Algorithm 3 walks
    from the root and emits the accepted CHILDREN (entries < 0 are emitted tokens without a tree node:
    skipped).  The root itself is the last token decoded before the step; Algorithm 3 needs
    Target(root, .), so the root is a query row of the verification pass and its K/V row (tree row 0) was
    computed in that pass too: with keep_root it stays in front of the accepted nodes whenever the
    walk emitted anything, so that the new prefix is old prefix + root + accepted path."""
    nodes = [int(a) for a in accepted_nodes if int(a) >= 0]
    if keep_root and len(accepted_nodes) > 0:
        nodes = [0] + nodes
    return nodes


def compact_kv(cache: np.ndarray, kv_row0: int, prefix_len: int, accepted_nodes: Sequence[int],
               keep_root: bool = False) -> int:
    """After a verification step the cache of a request holds prefix_len prefix rows followed by one row
    per tree node (node j at row kv_row0 + prefix_len + j).  The kept nodes k_0 < k_1 < ... (see
    kept_nodes) become part of the prefix: row kv_row0 + prefix_len + i takes the content of node k_i's
    row, in place.  Returns the new prefix length."""
    nodes = kept_nodes(accepted_nodes, keep_root)
    base = int(kv_row0) + int(prefix_len)
    gathered = [cache[base + a].copy() for a in nodes]       # all reads first: the definition is a gather
    for i, row in enumerate(gathered):
        cache[base + i] = row
    return int(prefix_len) + len(nodes)


# ----------------------------------------------------------------------------------------------------
# Paged KV cache (the paper is silent on the cache's memory layout; this is the layout a serving stack
# keeps its caches in).  The cache is a pool of pages of page_size rows.  Prefix token t of a request
# lies in the request's page number t // page_size, at row t % page_size of that page; the request's
# tree rows (one per node, in node order) are either a contiguous run of pool rows of their own, or
# (tree_row_offset / tree_row0 = None) tokens L, L + 1, ... of the same paged sequence.
# ----------------------------------------------------------------------------------------------------
def paged_prefix_rows(page_table_row: Sequence[int], page_size: int, length: int) -> List[int]:
    """Pool row of each of the first `length` tokens of a request whose pages are page_table_row."""
    return [int(page_table_row[t // page_size]) * page_size + t % page_size for t in range(int(length))]


def tree_attention_paged(q_bits, k_pool, v_pool, page_table, page_size: int, prefix_len, n_nodes, tree_row_offset,
                         parents_list, scale: float | None = None):
    """Tree-verify attention (same definition as tree_attention) with the prefix keys read through the
    page table and the tree keys from rows tree_row_offset[r] .. (tree_row_offset None: node j is token
    L + j of the paged sequence).  Returns float64 [sum n][H_q][D]."""
    outs = []
    qo = 0
    for r in range(len(prefix_len)):
        n, L = int(n_nodes[r]), int(prefix_len[r])
        if n:
            if tree_row_offset is None:
                rows = paged_prefix_rows(page_table[r], page_size, L + n)
            else:
                rows = paged_prefix_rows(page_table[r], page_size, L) + [int(tree_row_offset[r]) + j for j in range(n)]
            outs.append(tree_attention(q_bits[qo:qo + n], k_pool[rows], v_pool[rows], L, parents_list[r], scale))
        qo += n
    if not outs:
        return np.zeros((0,) + tuple(q_bits.shape[1:]), dtype=np.float64)
    return np.concatenate(outs, axis=0)


def compact_kv_paged(pool: np.ndarray, page_table_row: Sequence[int], page_size: int, tree_row0: int, prefix_len: int,
                     accepted_nodes: Sequence[int], keep_root: bool = False) -> int:
    """The kept nodes k_0 < k_1 < ... (see kept_nodes) become prefix tokens L, L + 1, ...: the pool row
    of token L + i (through the page table) takes the content of tree row tree_row0 + k_i (tree_row0 None:
    of token L + k_i, the node's row inside the paged sequence).  Returns the new prefix length."""
    nodes = kept_nodes(accepted_nodes, keep_root)
    L = int(prefix_len)
    dst = paged_prefix_rows(page_table_row, page_size, L + len(nodes))[L:]
    if tree_row0 is None:
        src = [int(page_table_row[(L + a) // page_size]) * page_size + (L + a) % page_size for a in nodes]
    else:
        src = [int(tree_row0) + a for a in nodes]
    gathered = [pool[s_].copy() for s_ in src]               # all reads first: the definition is a gather
    for d, row in zip(dst, gathered):
        pool[d] = row
    return L + len(nodes)
