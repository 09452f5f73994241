"""ctypes binding of libresps.so: the same entry points as include/resps.h, taking torch
tensors (device memory) and doing argument marshalling only -- every step of the path runs
in the library's CUDA kernels.  There is no CPU fallback: if the shared library cannot be
loaded, importing a symbol from here raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libresps.so")

RESPS_OK = 0
RESPS_ERR_INVALID_ARG = -1
RESPS_ERR_UNSUPPORTED_SHAPE = -2
RESPS_ERR_CAPACITY = -3
RESPS_ERR_CUDA = -4
RESPS_ERR_NO_DEVICE = -5
RESPS_STATUS_STEP_CLAMPED = 1
RESPS_STATUS_KV_OVERFLOW = 2
RESPS_STATUS_WAIT_TIMEOUT = 4
RESPS_STATUS_STALE_PLAN = 8
RESPS_DEBUG_ATTN_ROUNDS = 1
RESPS_DEBUG_ATTN_MIN_TILES = 2
RESPS_DEBUG_ATTN_STAGGER = 3
RESPS_DEBUG_SCAN_SLICES = 4
RESPS_DEBUG_ATTN_SINGLE = 5

EXPORTS = ("resps_create", "resps_destroy", "resps_strerror", "resps_status",
           "resps_workspace_bytes", "resps_debug_set", "resps_attention_replan", "resps_tree_expand", "resps_tree_expand_begin", "resps_tree_expand_level",
           "resps_tree_expand_finish", "resps_tree_attention",
           "resps_verify_accept", "resps_verify_accept_sampled", "resps_controller_step", "resps_scan_rows", "resps_row_scan_shard",
           "resps_tree_expand_merge", "resps_target_argmax_shard", "resps_verify_accept_merge", "resps_kv_compact", "resps_target_argmax_static")


class RespsShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_q_heads", "n_kv_heads", "head_dim", "vocab", "max_batch", "max_tt", "max_k",
                 "max_depth")]


class RespsPolicy(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("w1", "b1", "w2", "b2", "w3", "b3", "actions")] + \
               [(n, ctypes.c_int32) for n in ("n_features", "hidden", "n_actions")]


class RespsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def load() -> ctypes.CDLL:
    """Loads libresps.so (built in-tree by paper_2601_12212_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2601_12212_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
    lib.resps_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(RespsShape)]
    lib.resps_destroy.argtypes = [vp]
    lib.resps_strerror.argtypes = [i32]
    lib.resps_strerror.restype = ctypes.c_char_p
    lib.resps_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
    lib.resps_workspace_bytes.argtypes = [vp]
    lib.resps_workspace_bytes.restype = i64
    lib.resps_tree_expand.argtypes = [vp, vp, i32, vp, i64, i64, i64, i32, i32, vp,
                                      vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.resps_tree_expand_begin.argtypes = [vp, vp, i32, i32]
    lib.resps_tree_expand_level.argtypes = [vp, vp, i32, i32, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp]
    lib.resps_tree_expand_finish.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.resps_tree_attention.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, i64, i64, i64, i64,
                                         vp, f32, vp]
    lib.resps_verify_accept.argtypes = [vp, vp, vp, i32, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.resps_verify_accept_sampled.argtypes = [vp, vp, vp, i32, vp, i64, i64, vp, i64, i64, i64, f32, vp, vp, vp, vp,
                                                vp, vp, vp, vp, vp]
    lib.resps_controller_step.argtypes = [vp, ctypes.POINTER(RespsPolicy), vp, vp, vp, i64, i32, i32, f32, vp, vp, vp,
                                          vp, vp, vp, vp, vp, vp]
    lib.resps_scan_rows.argtypes = [vp]
    lib.resps_scan_rows.restype = i64
    lib.resps_row_scan_shard.argtypes = [vp, vp, i32, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp]
    lib.resps_tree_expand_merge.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                            vp, vp]
    lib.resps_target_argmax_shard.argtypes = [vp, vp, i32, vp, i64, i64, vp, vp]
    lib.resps_verify_accept_merge.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.resps_kv_compact.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, i32, i64, i64, i64, i64, vp]
    lib.resps_debug_set.argtypes = [vp, i32, i32]
    lib.resps_attention_replan.argtypes = [vp]
    lib.resps_target_argmax_static.argtypes = [vp, i32, i32, i32, vp, i64, i64, vp, vp]
    for name in EXPORTS:
        if name not in ("resps_strerror", "resps_workspace_bytes", "resps_scan_rows"):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().resps_strerror(int(code)).decode()


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _check(rc: int, where: str) -> None:
    if rc != RESPS_OK:
        raise RespsError(rc, where)


class Context:
    """Owns a resps_ctx (the library workspace) for one model shape on the current device."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, vocab: int,
                 max_batch: int = 1, max_tt: int = 128, max_k: int = 32, max_depth: int = 8):
        self.shape = RespsShape(n_q_heads, n_kv_heads, head_dim, vocab, max_batch, max_tt, max_k,
                                max_depth)
        self._h = ctypes.c_void_p()
        _check(load().resps_create(ctypes.byref(self._h), ctypes.byref(self.shape)), "resps_create")

    @property
    def handle(self):
        return self._h

    def workspace_bytes(self) -> int:
        return int(load().resps_workspace_bytes(self._h))

    def status(self, stream=None) -> int:
        out = ctypes.c_int32()
        _check(load().resps_status(self._h, _stream(stream), ctypes.byref(out)), "resps_status")
        return out.value

    def debug_set(self, key: int, value: int) -> None:
        """Test and tuning aid (see resps_debug_set in resps.h); never changes a result."""
        _check(load().resps_debug_set(self._h, int(key), int(value)), "resps_debug_set")

    def attention_replan(self) -> None:
        """The step parameters or node counts were changed behind the library's back: the next
        resps_tree_attention call derives its work list anew."""
        _check(load().resps_attention_replan(self._h), "resps_attention_replan")

    def close(self):
        if self._h:
            load().resps_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


STEP_DTYPE = torch.int32  # resps_step = 4 x int32 (tt, d, k, prefix_len): tensors of shape [batch, 4]


def resps_tree_expand(ctx: Context, steps, batch: int, draft_logits, ld_b: int, ld_level: int,
                      ld_row: int, n_levels: int, n_slots: int, root_token, tokens, parent, depth,
                      position_ids, mask, retrieve, n_leaves, n_nodes, stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_tree_expand(
        ctx.handle, _ptr(steps, i32), batch, _ptr(draft_logits, torch.float32), ld_b, ld_level, ld_row,
        n_levels, n_slots, _ptr(root_token, i32), _ptr(tokens, i32), _ptr(parent, i32),
        _ptr(depth, i32), _ptr(position_ids, i32), _ptr(mask), _ptr(retrieve, i32),
        _ptr(n_leaves, i32), _ptr(n_nodes, i32), _stream(stream)), "resps_tree_expand")


def resps_tree_expand_begin(ctx: Context, steps, batch: int, n_slots: int) -> None:
    _check(load().resps_tree_expand_begin(ctx.handle, _ptr(steps, torch.int32), batch, n_slots), "resps_tree_expand_begin")


def resps_tree_expand_level(ctx: Context, steps, batch: int, level: int, level_logits, ld_b: int, ld_row: int,
                            frontier_tokens, frontier_parent_slot, frontier_position_ids, frontier_node_index,
                            frontier_mask, frontier_score=None, stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_tree_expand_level(
        ctx.handle, _ptr(steps, i32), batch, level, _ptr(level_logits, torch.float32), ld_b, ld_row,
        _ptr(frontier_tokens, i32), _ptr(frontier_parent_slot, i32), _ptr(frontier_position_ids, i32),
        _ptr(frontier_node_index, i32), _ptr(frontier_mask), _ptr(frontier_score, torch.float64), _stream(stream)),
        "resps_tree_expand_level")


def resps_tree_expand_finish(ctx: Context, steps, batch: int, root_token, tokens, parent, depth, position_ids, mask,
                             retrieve, n_leaves, n_nodes, stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_tree_expand_finish(
        ctx.handle, _ptr(steps, i32), batch, _ptr(root_token, i32), _ptr(tokens, i32), _ptr(parent, i32),
        _ptr(depth, i32), _ptr(position_ids, i32), _ptr(mask), _ptr(retrieve, i32), _ptr(n_leaves, i32),
        _ptr(n_nodes, i32), _stream(stream)), "resps_tree_expand_finish")


def resps_tree_attention(ctx: Context, steps, n_nodes, batch: int, q, o, lse, k_cache, v_cache,
                         kv_stride_seq: int, kv_stride_head: int, kv_stride_tok: int,
                         kv_capacity: int, mask, softmax_scale: float, stream=None) -> None:
    i32, bf = torch.int32, torch.bfloat16
    _check(load().resps_tree_attention(
        ctx.handle, _ptr(steps, i32), _ptr(n_nodes, i32), batch, _ptr(q, bf), _ptr(o, bf),
        _ptr(lse, torch.float32), _ptr(k_cache, bf), _ptr(v_cache, bf), kv_stride_seq, kv_stride_head,
        kv_stride_tok, kv_capacity, _ptr(mask), float(softmax_scale), _stream(stream)),
        "resps_tree_attention")


def resps_verify_accept(ctx: Context, steps, n_nodes, batch: int, target_logits, ld_b: int,
                        ld_row: int, tokens, parent, target_argmax, accept_path, accept_len,
                        out_tokens, steps_next=None, stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_verify_accept(
        ctx.handle, _ptr(steps, i32), _ptr(n_nodes, i32), batch, _ptr(target_logits, torch.float32),
        ld_b, ld_row, _ptr(tokens, i32), _ptr(parent, i32), _ptr(target_argmax, i32),
        _ptr(accept_path, i32), _ptr(accept_len, i32), _ptr(out_tokens, i32), _ptr(steps_next, i32),
        _stream(stream)), "resps_verify_accept")


def resps_verify_accept_sampled(ctx: Context, steps, n_nodes, batch: int, target_logits, ld_b: int, ld_row: int,
                                draft_logits, draft_ld_b: int, draft_ld_level: int, draft_ld_row: int,
                                temperature: float, tokens, parent, u_accept, u_sample, accept_path, accept_len,
                                out_tokens, steps_next=None, stream=None) -> None:
    """Acceptance under sampling (T > 0) for the tree of the last resps_tree_expand on this context."""
    i32, f32, f64 = torch.int32, torch.float32, torch.float64
    _check(load().resps_verify_accept_sampled(
        ctx.handle, _ptr(steps, i32), _ptr(n_nodes, i32), batch, _ptr(target_logits, f32), ld_b, ld_row,
        _ptr(draft_logits, f32), draft_ld_b, draft_ld_level, draft_ld_row, float(temperature), _ptr(tokens, i32),
        _ptr(parent, i32), _ptr(u_accept, f64), _ptr(u_sample, f64), _ptr(accept_path, i32), _ptr(accept_len, i32),
        _ptr(out_tokens, i32), _ptr(steps_next, i32), _stream(stream)), "resps_verify_accept_sampled")


CONTROLLER_STATE_DTYPE = torch.int32  # resps_controller_state = (int32, int32, float32, int32): tensors [batch, 4]


def make_policy(w1, b1, w2, b2, w3, b3, actions) -> RespsPolicy:
    """Policy weights (fp32 CUDA tensors, [out][in]) and the action table (int32 [n_actions][3])."""
    f32 = torch.float32
    return RespsPolicy(_ptr(w1, f32), _ptr(b1, f32), _ptr(w2, f32), _ptr(b2, f32), _ptr(w3, f32), _ptr(b3, f32),
                       _ptr(actions, torch.int32), w1.shape[1], w1.shape[0], w3.shape[0])


def resps_controller_step(ctx: Context, policy: RespsPolicy, hidden_h, hidden_m, hidden_l, ld_hidden: int, batch: int,
                          interval: int, temperature: float, uniform, prev_accept_len, prev_elapsed_s, state, steps,
                          reward_avg, logits=None, action=None, stream=None) -> None:
    """One controller step (action cache, policy network, averaged reward); writes (TT, d, k) into `steps`."""
    bf, i32, f32 = torch.bfloat16, torch.int32, torch.float32
    _check(load().resps_controller_step(
        ctx.handle, ctypes.byref(policy), _ptr(hidden_h, bf), _ptr(hidden_m, bf), _ptr(hidden_l, bf), ld_hidden, batch,
        interval, float(temperature), _ptr(uniform, torch.float64), _ptr(prev_accept_len, i32),
        _ptr(prev_elapsed_s, f32), _ptr(state, i32), _ptr(steps, i32), _ptr(reward_avg, f32), _ptr(logits, f32),
        _ptr(action, i32), _stream(stream)), "resps_controller_step")


def resps_row_scan_shard(ctx: Context, steps, batch: int, draft_logits, ld_b: int, ld_level: int, ld_row: int,
                         n_levels: int, n_slots: int, part_val, part_id, part_lse, stream=None) -> None:
    _check(load().resps_row_scan_shard(
        ctx.handle, _ptr(steps, torch.int32), batch, _ptr(draft_logits, torch.float32), ld_b, ld_level, ld_row,
        n_levels, n_slots, _ptr(part_val, torch.float32), _ptr(part_id, torch.int32), _ptr(part_lse, torch.float64),
        _stream(stream)), "resps_row_scan_shard")


def resps_tree_expand_merge(ctx: Context, steps, batch: int, n_levels: int, n_slots: int, n_shards: int, all_val,
                            all_id, all_lse, shard_offset, root_token, tokens, parent, depth, position_ids, mask,
                            retrieve, n_leaves, n_nodes, stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_tree_expand_merge(
        ctx.handle, _ptr(steps, i32), batch, n_levels, n_slots, n_shards, _ptr(all_val, torch.float32),
        _ptr(all_id, i32), _ptr(all_lse, torch.float64), _ptr(shard_offset, i32), _ptr(root_token, i32),
        _ptr(tokens, i32), _ptr(parent, i32), _ptr(depth, i32), _ptr(position_ids, i32), _ptr(mask),
        _ptr(retrieve, i32), _ptr(n_leaves, i32), _ptr(n_nodes, i32), _stream(stream)), "resps_tree_expand_merge")


def resps_target_argmax_shard(ctx: Context, n_nodes, batch: int, target_logits, ld_b: int, ld_row: int, part_key,
                              stream=None) -> None:
    _check(load().resps_target_argmax_shard(
        ctx.handle, _ptr(n_nodes, torch.int32), batch, _ptr(target_logits, torch.float32), ld_b, ld_row,
        _ptr(part_key, torch.int64), _stream(stream)), "resps_target_argmax_shard")


def resps_verify_accept_merge(ctx: Context, steps, n_nodes, batch: int, n_shards: int, all_key, shard_offset, tokens,
                              parent, target_argmax, accept_path, accept_len, out_tokens, steps_next=None,
                              stream=None) -> None:
    i32 = torch.int32
    _check(load().resps_verify_accept_merge(
        ctx.handle, _ptr(steps, i32), _ptr(n_nodes, i32), batch, n_shards, _ptr(all_key, torch.int64),
        _ptr(shard_offset, i32), _ptr(tokens, i32), _ptr(parent, i32), _ptr(target_argmax, i32),
        _ptr(accept_path, i32), _ptr(accept_len, i32), _ptr(out_tokens, i32), _ptr(steps_next, i32),
        _stream(stream)), "resps_verify_accept_merge")


def shard_columns(vocab: int, n_shards: int, multiple: int = 4):
    """Column ranges [(offset, width)] of a vocabulary cut into n_shards pieces whose widths are multiples
    of `multiple` (the vectorised kernels want rows that start 16-byte aligned), the last taking the rest."""
    base = (vocab // n_shards) // multiple * multiple
    out, off = [], 0
    for p in range(n_shards):
        width = base if p < n_shards - 1 else vocab - off
        out.append((off, width))
        off += width
    return out


def all_gather_parts(parts, group=None):
    """All-gather of a rank's partial results (a list of tensors) over the ranks of a torch.distributed
    group: returns tensors with a leading [world] dimension, the layout the merge calls take."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = []
    for t in parts:
        pieces = [torch.empty_like(t) for _ in range(world)]
        dist.all_gather(pieces, t.contiguous(), group=group)
        out.append(torch.stack(pieces))
    return out


def resps_kv_compact(ctx: Context, steps, batch: int, accept_path, accept_len, k_cache_ptrs,
                     v_cache_ptrs, n_layers: int, kv_stride_seq: int, kv_stride_head: int,
                     kv_stride_tok: int, kv_capacity: int, steps_advanced: bool = False,
                     stream=None) -> None:
    """k_cache_ptrs / v_cache_ptrs: int64 CUDA tensors holding n_layers device pointers.
    steps_advanced: `steps` was already advanced by resps_verify_accept (steps_next aliased it)."""
    i32 = torch.int32
    _check(load().resps_kv_compact(
        ctx.handle, _ptr(steps, i32), int(bool(steps_advanced)), batch, _ptr(accept_path, i32),
        _ptr(accept_len, i32), _ptr(k_cache_ptrs, torch.int64), _ptr(v_cache_ptrs, torch.int64), n_layers,
        kv_stride_seq, kv_stride_head, kv_stride_tok, kv_capacity, _stream(stream)), "resps_kv_compact")


def resps_target_argmax_static(n_nodes, batch: int, max_tt: int, vocab: int, target_logits, ld_b: int,
                               ld_row: int, target_argmax, stream=None) -> None:
    """Per-node arg-max with no context and no allocation (scratch is a fixed array inside the
    library).  For callers that may not call cudaMalloc; batch * max_tt <= 1024."""
    i32 = torch.int32
    _check(load().resps_target_argmax_static(
        _ptr(n_nodes, i32), batch, max_tt, vocab, _ptr(target_logits, torch.float32), ld_b, ld_row,
        _ptr(target_argmax, i32), _stream(stream)), "resps_target_argmax_static")


def layer_pointer_table(caches: Sequence[torch.Tensor]) -> torch.Tensor:
    """Device array of the layers' base pointers, as resps_kv_compact expects."""
    return torch.tensor([c.data_ptr() for c in caches], dtype=torch.int64, device=caches[0].device)
