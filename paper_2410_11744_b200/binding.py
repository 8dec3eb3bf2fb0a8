"""Thin ctypes binding of libdyspec.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/dyspec.h) and passes raw
device pointers of torch tensors plus the current CUDA stream.  All arithmetic happens in the CUDA
kernels of the library; there is no fallback: if the library has not been built, importing this
module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdyspec.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2410_11744_b200.build` "
        "(there is no CPU or PyTorch fallback for the CUDA path)")

lib = ctypes.CDLL(LIB_PATH)

_c = ctypes
_vp, _i32, _i64, _sz, _f32 = _c.c_void_p, _c.c_int, _c.c_int64, _c.c_size_t, _c.c_float

# name -> (restype, argtypes); mirrors include/dyspec.h one to one
SIGNATURES = {
    "dyspec_error_string": (_c.c_char_p, [_i32]),
    "dyspec_version": (_i32, []),
    "dyspec_words_per_row": (_i32, [_i32]),
    "dyspec_set_tuning": (_i32, [_i32, _i32, _i32]),
    "dyspec_set_trace": (_i32, [_vp, _i32]),
    "dyspec_build_tree_mask": (_i32, [_vp, _i32, _vp, _vp, _i32, _vp, _vp]),
    "dyspec_build_tree_mask_batched": (_i32, [_vp, _vp, _i32, _vp, _vp, _i32, _vp, _vp]),
    "dyspec_plan_create": (_i32, [_c.POINTER(_vp), _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i64, _i32, _f32]),
    "dyspec_plan_destroy": (_i32, [_vp]),
    "dyspec_plan_workspace_bytes": (_sz, [_vp]),
    "dyspec_plan_info": (_i64, [_vp, _i32]),
    "dyspec_schedule_dry_run": (_i32, [_i32, _i32, _i32, _i32, _vp, _vp, _i32, _vp, _i32, _vp, _i32, _vp]),
    "dyspec_plan_build_tree_mask": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_tree_attention_ragged": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "dyspec_set_default_shape": (_i32, [_i32, _i32, _i32, _i32, _f32]),
    "dyspec_tree_attention": (_i32, [_vp, _vp, _vp, _i32, _vp, _i32, _vp, _vp]),
    "dyspec_dfs_reorder": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_plan_dfs_reorder": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_build_tree_mask_tiles": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _vp, _vp]),
    "dyspec_plan_build_tree_mask_tiles": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_mask_block_count": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp]),
    "dyspec_tree_attention_ragged_sparse": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "dyspec_verify_tree": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp, _vp]),
    "dyspec_build_tree_greedy": (_i32, [_vp, _i32, _i32, _vp, _i32, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_build_tree_threshold": (_i32, [_vp, _i32, _i32, _vp, _i32, _vp, _i32, _f32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dyspec_compact_kv": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp]),
    "dyspec_plan_create_paged": (_i32, [_c.POINTER(_vp), _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i64, _i32, _i32, _f32]),
    "dyspec_tree_attention_paged": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "dyspec_compact_kv_paged": (_i32, [_vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp]),
    "dyspec_release_cache": (_i32, []),
    "dyspec_tree_attention_static": (_i32, [_vp, _vp, _vp, _i32, _vp, _i32, _vp, _i32, _i32, _i32, _i32, _f32, _vp, _vp]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class DyspecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {dyspec_error_string(code)} ({code})")


def _check(code: int, where: str) -> None:
    if code != 0:
        raise DyspecError(code, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream=None) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def dyspec_error_string(code: int) -> str:
    return lib.dyspec_error_string(code).decode()


def dyspec_version() -> int:
    return lib.dyspec_version()


def dyspec_words_per_row(max_nodes: int) -> int:
    return lib.dyspec_words_per_row(max_nodes)


def dyspec_set_tuning(force_regime: int = -1, force_ctas: int = 0, combine_mode: int = 2) -> None:
    _check(lib.dyspec_set_tuning(force_regime, force_ctas, combine_mode), "dyspec_set_tuning")


def dyspec_set_trace(trace_buffer=None, capacity_entries: int = 0) -> None:
    _check(lib.dyspec_set_trace(_ptr(trace_buffer), capacity_entries), "dyspec_set_trace")


def dyspec_build_tree_mask(parents, n_nodes: int, ancestor_bits, depths=None, words_per_row: int = 0,
                           status=None, stream=None) -> None:
    """parents: int32 device tensor [n]; ancestor_bits: int32/uint32 device tensor [n][W]; depths: int32 [n] or None."""
    _check(lib.dyspec_build_tree_mask(_ptr(parents), n_nodes, _ptr(ancestor_bits), _ptr(depths), words_per_row,
                                      _ptr(status), _stream(stream)), "dyspec_build_tree_mask")


class Plan:
    """Owns a dyspec_plan_t*: static shape + ragged batch structure + scheduled work list."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, prefix_len: Sequence[int],
                 n_nodes: Sequence[int], kv_row_offset: Sequence[int], kv_total_rows: int, words_per_row: int,
                 scale: float = 0.0, page_size: Optional[int] = None):
        """A page_size makes a plan for the paged cache: kv_row_offset is then the first tree row of each
        request and kv_total_rows the rows of the pool (dyspec_plan_create_paged)."""
        n_req = len(prefix_len)
        pl = (_c.c_int32 * max(1, n_req))(*[int(x) for x in prefix_len])
        nn = (_c.c_int32 * max(1, n_req))(*[int(x) for x in n_nodes])
        off = None if kv_row_offset is None else (_c.c_int64 * max(1, n_req))(*[int(x) for x in kv_row_offset])
        handle = _vp()
        if page_size is not None:
            # kv_row_offset None: the tree rows are tokens L .. L + n - 1 of the paged sequence (NULL in the C call)
            _check(lib.dyspec_plan_create_paged(_c.byref(handle), n_q_heads, n_kv_heads, head_dim, n_req,
                                                _c.cast(pl, _vp), _c.cast(nn, _vp),
                                                _vp() if off is None else _c.cast(off, _vp), int(kv_total_rows),
                                                int(page_size), words_per_row, float(scale)), "dyspec_plan_create_paged")
        else:
            _check(lib.dyspec_plan_create(_c.byref(handle), n_q_heads, n_kv_heads, head_dim, n_req,
                                          _c.cast(pl, _vp), _c.cast(nn, _vp), _c.cast(off, _vp), int(kv_total_rows),
                                          words_per_row, float(scale)), "dyspec_plan_create")
        self.handle = handle
        self.page_size = int(page_size or 0)
        self.words_per_row = words_per_row
        self.total_nodes = int(sum(int(x) for x in n_nodes))

    def workspace_bytes(self) -> int:
        return int(lib.dyspec_plan_workspace_bytes(self.handle))

    def info(self, field: int) -> int:
        return int(lib.dyspec_plan_info(self.handle, field))

    def describe(self) -> dict:
        names = ["items", "ctas", "groups", "split_groups", "max_splits", "regime", "key_tiles", "rows_per_tile",
                 "cluster", "dynamic", "combine_launch"]
        return {k: self.info(i) for i, k in enumerate(names)}

    def destroy(self) -> None:
        if self.handle:
            lib.dyspec_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def dyspec_plan_create(*args, **kwargs) -> Plan:
    return Plan(*args, **kwargs)


def dyspec_plan_create_paged(n_q_heads: int, n_kv_heads: int, head_dim: int, prefix_len: Sequence[int],
                             n_nodes: Sequence[int], tree_row_offset: Sequence[int], kv_total_rows: int, page_size: int,
                             words_per_row: int, scale: float = 0.0) -> Plan:
    return Plan(n_q_heads, n_kv_heads, head_dim, prefix_len, n_nodes, tree_row_offset, kv_total_rows, words_per_row,
                scale, page_size=page_size)


def dyspec_plan_destroy(plan: Plan) -> None:
    plan.destroy()


def dyspec_plan_workspace_bytes(plan: Plan) -> int:
    return plan.workspace_bytes()


def dyspec_plan_info(plan: Plan, field: int) -> int:
    return plan.info(field)


def dyspec_schedule_dry_run(n_q_heads: int, n_kv_heads: int, head_dim: int, prefix_len: Sequence[int],
                            n_nodes: Sequence[int], words_per_row: int, max_items: int = 1 << 16):
    """Host-only scheduler run -> (items int32 [n][8], cta_begin int32 [n_ctas + 1], info dict)."""
    import numpy as np
    n_req = len(prefix_len)
    pl = np.asarray(list(prefix_len) or [0], dtype=np.int32)
    nn = np.asarray(list(n_nodes) or [0], dtype=np.int32)
    items = np.zeros((max_items, 8), dtype=np.int32)
    cta = np.zeros(max_items + 1, dtype=np.int32)
    info = np.zeros(12, dtype=np.int64)
    rc = lib.dyspec_schedule_dry_run(n_q_heads, n_kv_heads, head_dim, n_req, pl.ctypes.data, nn.ctypes.data,
                                     words_per_row, items.ctypes.data, max_items, cta.ctypes.data, max_items + 1,
                                     info.ctypes.data)
    if rc < 0:
        raise DyspecError(rc, "dyspec_schedule_dry_run")
    if rc > max_items:
        return dyspec_schedule_dry_run(n_q_heads, n_kv_heads, head_dim, prefix_len, n_nodes, words_per_row, rc)
    names = ["items", "ctas", "groups", "split_groups", "max_splits", "regime", "key_tiles", "rows_per_tile",
             "keys_per_tile", "workspace_bytes", "cluster", "combine_launch"]
    d = {k: int(v) for k, v in zip(names, info)}
    return items[:rc].copy(), cta[:d["ctas"] + 1].copy(), d


def dyspec_plan_build_tree_mask(plan: Plan, parents, ancestor_bits, depths=None, status=None, stream=None) -> None:
    _check(lib.dyspec_plan_build_tree_mask(plan.handle, _ptr(parents), _ptr(ancestor_bits), _ptr(depths),
                                           _ptr(status), _stream(stream)), "dyspec_plan_build_tree_mask")


def dyspec_tree_attention_ragged(plan: Plan, q, k_cache, v_cache, ancestor_bits, out, workspace=None,
                                 workspace_bytes: Optional[int] = None, status=None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dyspec_tree_attention_ragged(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ancestor_bits),
                                            _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status),
                                            _stream(stream)), "dyspec_tree_attention_ragged")


def dyspec_set_default_shape(n_q_heads: int, n_kv_heads: int, head_dim: int, words_per_row: int,
                             scale: float = 0.0) -> None:
    _check(lib.dyspec_set_default_shape(n_q_heads, n_kv_heads, head_dim, words_per_row, float(scale)),
           "dyspec_set_default_shape")


def dyspec_tree_attention(q, k_cache, v_cache, prefix_len: int, ancestor_bits, n_nodes: int, out, stream=None) -> None:
    _check(lib.dyspec_tree_attention(_ptr(q), _ptr(k_cache), _ptr(v_cache), prefix_len, _ptr(ancestor_bits), n_nodes,
                                     _ptr(out), _stream(stream)), "dyspec_tree_attention")


def dyspec_tree_attention_static(q, k_cache, v_cache, prefix_len: int, ancestor_bits, n_nodes: int, out, n_q_heads: int,
                                 n_kv_heads: int, head_dim: int, words_per_row: int, scale: float = 0.0, status=None,
                                 stream=None) -> None:
    """Single-request attention for callers that may not allocate device memory: the work list and the
    split-KV partials go into the library's fixed device array (16 MiB, shared by all calls)."""
    _check(lib.dyspec_tree_attention_static(_ptr(q), _ptr(k_cache), _ptr(v_cache), prefix_len, _ptr(ancestor_bits),
                                            n_nodes, _ptr(out), n_q_heads, n_kv_heads, head_dim, words_per_row,
                                            float(scale), _ptr(status), _stream(stream)),
           "dyspec_tree_attention_static")


def dyspec_dfs_reorder(parents, n_nodes: int, order=None, new_of_old=None, new_parents=None, status=None,
                       stream=None) -> None:
    """Depth-first renumbering of one tree; all arrays are int32 device tensors [n] (outputs may be None)."""
    _check(lib.dyspec_dfs_reorder(_ptr(parents), n_nodes, _ptr(order), _ptr(new_of_old), _ptr(new_parents),
                                  _ptr(status), _stream(stream)), "dyspec_dfs_reorder")


def dyspec_plan_dfs_reorder(plan: Plan, parents, order=None, new_of_old=None, new_parents=None, status=None,
                            stream=None) -> None:
    _check(lib.dyspec_plan_dfs_reorder(plan.handle, _ptr(parents), _ptr(order), _ptr(new_of_old), _ptr(new_parents),
                                       _ptr(status), _stream(stream)), "dyspec_plan_dfs_reorder")


def dyspec_build_tree_mask_tiles(parents, n_nodes: int, ancestor_bits, depths, node_tiles, words_per_row: int,
                                 status=None, stream=None) -> None:
    _check(lib.dyspec_build_tree_mask_tiles(_ptr(parents), n_nodes, _ptr(ancestor_bits), _ptr(depths), _ptr(node_tiles),
                                            words_per_row, _ptr(status), _stream(stream)),
           "dyspec_build_tree_mask_tiles")


def dyspec_plan_build_tree_mask_tiles(plan: Plan, parents, ancestor_bits, depths, node_tiles, status=None,
                                      stream=None) -> None:
    _check(lib.dyspec_plan_build_tree_mask_tiles(plan.handle, _ptr(parents), _ptr(ancestor_bits), _ptr(depths),
                                                 _ptr(node_tiles), _ptr(status), _stream(stream)),
           "dyspec_plan_build_tree_mask_tiles")


def dyspec_mask_block_count(ancestor_bits, n_nodes: int, words_per_row: int, block: int, count, stream=None) -> None:
    """count: int64 device tensor [1] (written)."""
    _check(lib.dyspec_mask_block_count(_ptr(ancestor_bits), n_nodes, words_per_row, block, _ptr(count),
                                       _stream(stream)), "dyspec_mask_block_count")


def dyspec_tree_attention_ragged_sparse(plan: Plan, q, k_cache, v_cache, ancestor_bits, node_tiles, out, workspace=None,
                                        workspace_bytes: Optional[int] = None, status=None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dyspec_tree_attention_ragged_sparse(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                                   _ptr(ancestor_bits), _ptr(node_tiles), _ptr(out), _ptr(workspace),
                                                   workspace_bytes, _ptr(status), _stream(stream)),
           "dyspec_tree_attention_ragged_sparse")


def dyspec_verify_tree(parents, tokens, draft_probs, target_probs, accept_u, sample_u, node_offsets, n_req: int,
                       max_nodes: int, vocab: int, accepted_tokens, accepted_nodes, n_accepted, max_out: int,
                       bonus_at_leaf: bool = False, status=None, stream=None) -> None:
    """Tree verification (Algorithm 3) for n_req requests; all arrays are device tensors (see include/dyspec.h)."""
    _check(lib.dyspec_verify_tree(_ptr(parents), _ptr(tokens), _ptr(draft_probs), _ptr(target_probs), _ptr(accept_u),
                                  _ptr(sample_u), _ptr(node_offsets), n_req, max_nodes, vocab, int(bool(bonus_at_leaf)),
                                  _ptr(accepted_tokens), _ptr(accepted_nodes), _ptr(n_accepted), max_out, _ptr(status),
                                  _stream(stream)), "dyspec_verify_tree")


def dyspec_build_tree_greedy(draft_table, n_rows: int, vocab: int, uniforms, n_uniforms: int, root_row, n_req: int, m: int,
                             parents, tokens, values, child_values, rows, n_nodes, stream=None) -> None:
    """Algorithm 1 over a table-lookup draft model; outputs are device tensors [n_req][m + 1] (see include/dyspec.h)."""
    _check(lib.dyspec_build_tree_greedy(_ptr(draft_table), n_rows, vocab, _ptr(uniforms), n_uniforms, _ptr(root_row), n_req,
                                        m, _ptr(parents), _ptr(tokens), _ptr(values), _ptr(child_values), _ptr(rows),
                                        _ptr(n_nodes), _stream(stream)), "dyspec_build_tree_greedy")


def dyspec_build_tree_threshold(draft_table, n_rows: int, vocab: int, uniforms, n_uniforms: int, root_row, n_req: int,
                                threshold: float, max_nodes: int, parents, tokens, values, child_values, rows, n_nodes,
                                stream=None) -> None:
    """Algorithm 2 over a table-lookup draft model; outputs are device tensors [n_req][max_nodes + 1]."""
    _check(lib.dyspec_build_tree_threshold(_ptr(draft_table), n_rows, vocab, _ptr(uniforms), n_uniforms, _ptr(root_row),
                                           n_req, float(threshold), max_nodes, _ptr(parents), _ptr(tokens), _ptr(values),
                                           _ptr(child_values), _ptr(rows), _ptr(n_nodes), _stream(stream)),
           "dyspec_build_tree_threshold")


def dyspec_compact_kv(k_cache, v_cache, kv_row_offset, prefix_len, accepted_nodes, n_accepted, n_req: int, max_out: int,
                      n_kv_heads: int, head_dim: int, new_prefix_len=None, stream=None, keep_root: bool = False) -> None:
    """Moves the accepted nodes' K/V rows behind the prefix, in place (see include/dyspec.h)."""
    _check(lib.dyspec_compact_kv(_ptr(k_cache), _ptr(v_cache), _ptr(kv_row_offset), _ptr(prefix_len), _ptr(accepted_nodes),
                                 _ptr(n_accepted), n_req, max_out, n_kv_heads, head_dim, int(bool(keep_root)),
                                 _ptr(new_prefix_len), _stream(stream)), "dyspec_compact_kv")


def dyspec_tree_attention_paged(plan: Plan, q, k_cache, v_cache, page_table, pages_per_req: int, ancestor_bits,
                                node_tiles, out, workspace=None, status=None, stream=None) -> None:
    """Tree attention over a paged cache (see include/dyspec.h); node_tiles may be None."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dyspec_tree_attention_paged(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(page_table),
                                           int(pages_per_req), _ptr(ancestor_bits), _ptr(node_tiles), _ptr(out),
                                           _ptr(workspace), ws_bytes, _ptr(status), _stream(stream)),
           "dyspec_tree_attention_paged")


def dyspec_compact_kv_paged(k_cache, v_cache, tree_row_offset, page_table, pages_per_req: int, page_size: int, prefix_len,
                            accepted_nodes, n_accepted, n_req: int, max_out: int, n_kv_heads: int, head_dim: int,
                            new_prefix_len=None, status=None, stream=None, keep_root: bool = False) -> None:
    """Moves the accepted nodes' K/V rows from the tree rows into the prefix pages (see include/dyspec.h)."""
    _check(lib.dyspec_compact_kv_paged(_ptr(k_cache), _ptr(v_cache), _ptr(tree_row_offset), _ptr(page_table),
                                       int(pages_per_req), int(page_size), _ptr(prefix_len), _ptr(accepted_nodes),
                                       _ptr(n_accepted), n_req, max_out, n_kv_heads, head_dim, int(bool(keep_root)),
                                       _ptr(new_prefix_len), _ptr(status), _stream(stream)), "dyspec_compact_kv_paged")


def dyspec_release_cache() -> None:
    """Frees what dyspec_tree_attention cached (see include/dyspec.h)."""
    _check(lib.dyspec_release_cache(), "dyspec_release_cache")


def dyspec_build_tree_mask_batched(parents, node_offsets: Sequence[int], ancestor_bits, depths, words_per_row: int,
                                   status=None, stream=None) -> None:
    """Ragged batch without a plan: node_offsets is a host sequence [n_req + 1] (see include/dyspec.h)."""
    n_req = len(node_offsets) - 1
    offs = (_c.c_int32 * (n_req + 1))(*[int(x) for x in node_offsets])
    _check(lib.dyspec_build_tree_mask_batched(_ptr(parents), _c.cast(offs, _vp), n_req, _ptr(ancestor_bits), _ptr(depths),
                                              words_per_row, _ptr(status), _stream(stream)), "dyspec_build_tree_mask_batched")
