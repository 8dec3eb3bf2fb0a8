"""Device-side harness around the binding: holds one ragged batch on the GPU and runs the hot path on it.

Only plumbing (torch for device memory and streams); every step of the path is a library call.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from .workloads import Workload


def _bits_to_bf16(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DeviceBatch:
    """Buffers + plan for one Workload.  `step()` = mask build + attention (+ combine) on the current stream."""

    def __init__(self, w: Workload, device="cuda:0", words_per_row: int | None = None, upload: bool = True,
                 plan: "B.Plan | None" = None, sparse: bool = False, paged=None):
        """paged: a workloads.PagedWorkload of w; the cache buffers are then its pool and the attention
        reads the prefix through its page table."""
        self.w = w
        self.paged = paged
        self.sparse = sparse            # also emit per-node tile sets and let the attention skip empty tree tiles
        self.device = torch.device(device)
        max_n = int(w.n_nodes.max()) if w.n_req else 0
        self.W = words_per_row or B.dyspec_words_per_row(max_n)
        self.total_nodes = w.total_nodes
        self.kv_total_rows = int(w.k.shape[0]) if paged is None else paged.pool_rows
        # a plan depends only on the batch structure, so buffers with the same structure can share one
        if plan is None and paged is not None:
            plan = B.Plan(w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len, w.n_nodes, paged.tree_row_offset,
                          self.kv_total_rows, self.W, 0.0, page_size=paged.page_size)
        self.plan = plan or B.Plan(w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len, w.n_nodes, w.kv_row_offset,
                                   self.kv_total_rows, self.W, 0.0)
        dev = self.device
        n = max(1, self.total_nodes)
        self.bits = torch.zeros((n, self.W), dtype=torch.int32, device=dev)
        self.depths = torch.zeros((n,), dtype=torch.int32, device=dev)
        self.node_tiles = torch.zeros((n,), dtype=torch.int32, device=dev) if sparse else None
        self.status = torch.zeros((1,), dtype=torch.int32, device=dev)
        self.out = torch.zeros((n, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        ws = self.plan.workspace_bytes()
        self.workspace = torch.zeros((max(ws, 256),), dtype=torch.uint8, device=dev)   # zeroed once: queue words live in it
        self.workspace_bytes = ws
        if upload:
            self.upload()

    def upload(self):
        w, dev = self.w, self.device
        self.parents = torch.from_numpy(w.parents_concat if self.total_nodes else np.zeros(1, np.int32)).to(dev)
        self.q = _bits_to_bf16(w.q if self.total_nodes else np.zeros((1, w.n_q_heads, w.head_dim), np.uint16), dev)
        kv_shape = (max(1, self.kv_total_rows), w.n_kv_heads, w.head_dim)
        src = w if self.paged is None else self.paged
        self.k = _bits_to_bf16(src.k if self.kv_total_rows else np.zeros(kv_shape, np.uint16), dev)
        self.v = _bits_to_bf16(src.v if self.kv_total_rows else np.zeros(kv_shape, np.uint16), dev)
        if self.paged is not None:
            self.page_table = torch.from_numpy(np.ascontiguousarray(self.paged.page_table)).to(dev)

    def build_mask(self):
        if self.sparse:
            B.dyspec_plan_build_tree_mask_tiles(self.plan, self.parents, self.bits, self.depths, self.node_tiles,
                                                self.status)
        else:
            B.dyspec_plan_build_tree_mask(self.plan, self.parents, self.bits, self.depths, self.status)

    def attention(self):
        if self.paged is not None:
            B.dyspec_tree_attention_paged(self.plan, self.q, self.k, self.v, self.page_table, self.paged.pages_per_req,
                                          self.bits, self.node_tiles if self.sparse else None, self.out,
                                          self.workspace, self.status)
        elif self.sparse:
            B.dyspec_tree_attention_ragged_sparse(self.plan, self.q, self.k, self.v, self.bits, self.node_tiles,
                                                  self.out, self.workspace, self.workspace_bytes, self.status)
        else:
            B.dyspec_tree_attention_ragged(self.plan, self.q, self.k, self.v, self.bits, self.out, self.workspace,
                                           self.workspace_bytes, self.status)

    def dfs_reorder(self):
        """Runs the reorder kernel on the batch's parents -> (order, new_of_old, new_parents) int32 numpy [sum n]."""
        n = max(1, self.total_nodes)
        order = torch.full((n,), -7, dtype=torch.int32, device=self.device)
        new_of_old = torch.full((n,), -7, dtype=torch.int32, device=self.device)
        new_parents = torch.full((n,), -7, dtype=torch.int32, device=self.device)
        B.dyspec_plan_dfs_reorder(self.plan, self.parents, order, new_of_old, new_parents, self.status)
        torch.cuda.synchronize(self.device)
        m = self.total_nodes
        return order[:m].cpu().numpy(), new_of_old[:m].cpu().numpy(), new_parents[:m].cpu().numpy()

    def step(self):
        self.build_mask()
        self.attention()

    def results(self):
        """(ancestor_bits uint32 [n][W], depths int32 [n], out bf16 bits uint16 [n][Hq][D], status int)."""
        torch.cuda.synchronize(self.device)
        n = self.total_nodes
        bits = self.bits[:n].cpu().numpy().view(np.uint32)
        depths = self.depths[:n].cpu().numpy()
        out = bf16_tensor_to_bits(self.out[:n])
        return bits, depths, out, int(self.status.item())
