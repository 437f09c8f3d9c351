"""ctypes binding of the CUDA C-ABI library (`include/hsd.h`), same function names, argument marshalling only.

Pointer arguments accept a torch tensor (its `data_ptr()` is passed), an int address or None.  Every
function returns the library's status; `check()` turns a non-zero status into `HsdError`.  There is no CPU
fallback: importing this module raises if the built library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhsd.so")

HSD_OK = 0
HSD_ERR_INVALID_ARG, HSD_ERR_SHAPE, HSD_ERR_TOO_LONG, HSD_ERR_WORKSPACE = -1, -2, -3, -4
HSD_ERR_KV_CAPACITY, HSD_ERR_CUDA, HSD_ERR_DEVICE_CHECK, HSD_ERR_NO_DEVICE = -5, -6, -7, -8
HSD_MAX_Q_LEN = 4097
HSD_MAX_TREE_ROWS = 128
HSD_MAX_WINDOW = 8
HSD_DSV_MAX_CANDIDATES = 64
HSD_KV_BLOCK = 64
HSD_FLAG_SIMT_DEBUG = 1
HSD_FLAG_SIMT_ATTENTION = 2
HSD_FLAG_DETERMINISTIC = 4
HSD_FLAG_NO_PDL = 8
HSD_FLAG_NO_PAIR = 16
HSD_FLAG_NO_HOST_GRAPH = 32
HSD_NOALLOC_MAX_ROWS = 8192

EXPORTS = [
    "hsd_status_string", "hsd_create", "hsd_destroy", "hsd_workspace_bytes", "hsd_prefill", "hsd_verify_regions",
    "hsd_verify_page", "hsd_kv_commit", "hsd_verify_regions_host", "hsd_device_status", "hsd_last_cuda_error", "hsd_launch_count",
    "hsd_profile_enable", "hsd_profile_read", "hsd_debug_logits", "hsd_debug_buffer", "hsd_op_linear",
    "hsd_op_lm_head_argmax", "hsd_op_lm_head_argmax_noalloc", "hsd_debug_set_gemm_tile", "hsd_debug_set_attn_plan",
    "hsd_verify_tree", "hsd_kv_commit_tree", "hsd_dsv_build", "hsd_debug_tap", "hsd_stage_begin", "hsd_stage_advance",
    "hsd_stage_aggregate",
]
HSD_TAP_X, HSD_TAP_H_ATTN, HSD_TAP_H_FFN, HSD_TAP_Q, HSD_TAP_ATTN, HSD_TAP_ACT, HSD_TAP_X_MID = range(7)


class HsdError(RuntimeError):
    def __init__(self, status: int, what: str = ""):
        self.status = status
        msg = _lib.hsd_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{what}: {msg} ({status})" if what else f"{msg} ({status})")


class hsd_model_config(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("d_ffn", C.c_int), ("vocab", C.c_int), ("rope_base", C.c_float),
                ("rms_eps", C.c_float), ("kv_block", C.c_int), ("flags", C.c_int), ("qk_norm", C.c_int)]


class hsd_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("w_qkv", C.POINTER(C.c_void_p)),
                ("w_o", C.POINTER(C.c_void_p)), ("ffn_norm", C.POINTER(C.c_void_p)),
                ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
                ("q_norm", C.POINTER(C.c_void_p)), ("k_norm", C.POINTER(C.c_void_p))]


class hsd_kv(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("n_blocks", C.c_int),
                ("block_table", C.c_void_p), ("max_blocks_per_seq", C.c_int), ("seq_lens", C.c_void_p),
                ("n_slots", C.c_int)]


class hsd_stage(C.Structure):
    _fields_ = [("n_lanes", C.c_int), ("n_seqs", C.c_int), ("window_n", C.c_int), ("out_stride", C.c_int),
                ("idle_slot", C.c_int), ("lane_seq", C.c_void_p), ("lane_slot", C.c_void_p), ("window", C.c_void_p),
                ("first_token", C.c_void_p), ("seq_slot", C.c_void_p), ("max_new", C.c_void_p),
                ("out_tokens", C.c_void_p), ("out_len", C.c_void_p), ("seq_steps", C.c_void_p),
                ("seq_accepted", C.c_void_p), ("counters", C.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_12957_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    lib.hsd_status_string.restype = C.c_char_p
    lib.hsd_status_string.argtypes = [i]
    lib.hsd_create.argtypes = [C.POINTER(hsd_model_config), C.POINTER(hsd_weights), C.POINTER(vp)]
    lib.hsd_destroy.argtypes = [vp]
    lib.hsd_workspace_bytes.restype = sz
    lib.hsd_workspace_bytes.argtypes = [vp, i, i]
    lib.hsd_prefill.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, vp, i, i, vp, vp, sz, vp]
    lib.hsd_verify_regions.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, i, i, f, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.hsd_verify_page.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, i, f, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.hsd_kv_commit.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, vp]
    lib.hsd_verify_tree.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, vp, i, i, f, vp, vp, vp, vp, vp, vp, vp, vp, sz,
                                    vp]
    lib.hsd_kv_commit_tree.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, i, vp, vp]
    lib.hsd_dsv_build.argtypes = [vp, i, i, vp, vp, vp, i, vp, i, vp, i, vp, i, vp, vp, vp, vp, vp, i, vp]
    lib.hsd_stage_begin.argtypes = [vp, C.POINTER(hsd_stage), C.POINTER(hsd_kv), vp]
    lib.hsd_stage_advance.argtypes = [vp, C.POINTER(hsd_stage), C.POINTER(hsd_kv), vp, vp, vp, i, vp]
    lib.hsd_stage_aggregate.argtypes = [vp, C.POINTER(hsd_stage), vp, i, vp, vp]
    lib.hsd_verify_regions_host.argtypes = [vp, C.POINTER(hsd_kv), i, vp, vp, vp, f, i, vp, vp, vp, C.POINTER(C.c_int), vp, sz, vp]
    lib.hsd_device_status.argtypes = [vp, vp, vp, C.POINTER(C.c_int)]
    lib.hsd_last_cuda_error.argtypes = [vp]
    lib.hsd_launch_count.restype = C.c_longlong
    lib.hsd_launch_count.argtypes = [vp]
    lib.hsd_profile_enable.argtypes = [vp, i]
    lib.hsd_profile_read.argtypes = [vp, i, C.POINTER(C.c_char_p), C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
    lib.hsd_debug_logits.argtypes = [vp, vp, i, i, vp, vp]
    lib.hsd_debug_buffer.argtypes = [vp, vp, i, i, C.c_char_p, C.POINTER(vp), C.POINTER(sz)]
    lib.hsd_debug_tap.argtypes = [vp, i, i, vp, sz]
    lib.hsd_debug_set_gemm_tile.argtypes = [vp, i, i]
    lib.hsd_debug_set_attn_plan.argtypes = [vp, i, i]
    lib.hsd_op_linear.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
    lib.hsd_op_lm_head_argmax.argtypes = [vp, vp, i, vp, vp, sz, vp, vp, vp, vp]
    lib.hsd_op_lm_head_argmax_noalloc.argtypes = [vp, vp, i, vp, vp, vp, vp, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("hsd_status_string", "hsd_workspace_bytes", "hsd_launch_count"):
            fn.restype = i
    return lib


_lib = None
_lib = _load()


def _p(x):
    if x is None:
        return None
    if isinstance(x, int):
        return C.c_void_p(x)
    return C.c_void_p(x.data_ptr())


def check(status: int, what: str = "") -> int:
    if status != HSD_OK:
        raise HsdError(status, what)
    return status


def make_config(cfg, flags: int = 0) -> hsd_model_config:
    return hsd_model_config(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                            cfg.vocab, cfg.rope_base, cfg.rms_eps, cfg.kv_block, flags,
                            1 if getattr(cfg, "qk_norm", False) else 0)


def make_weights(embed, lm_head, final_norm, attn_norm: Sequence, w_qkv: Sequence, w_o: Sequence,
                 ffn_norm: Sequence, w_gate_up: Sequence, w_down: Sequence, q_norm: Optional[Sequence] = None,
                 k_norm: Optional[Sequence] = None) -> hsd_weights:
    def arr(ts):
        a = (C.c_void_p * len(ts))(*[t.data_ptr() if t is not None else None for t in ts])
        return a
    w = hsd_weights()
    w.embed, w.lm_head, w.final_norm = embed.data_ptr(), lm_head.data_ptr(), final_norm.data_ptr()
    keep = []
    for name, ts in (("attn_norm", attn_norm), ("w_qkv", w_qkv), ("w_o", w_o), ("ffn_norm", ffn_norm),
                     ("w_gate_up", w_gate_up), ("w_down", w_down), ("q_norm", q_norm), ("k_norm", k_norm)):
        if ts is None:
            continue
        a = arr(ts)
        keep.append(a)
        setattr(w, name, C.cast(a, C.POINTER(C.c_void_p)))
    w._keep = keep          # the pointer arrays must outlive hsd_create
    return w


def make_kv(k_pool, v_pool, n_blocks: int, block_table, max_blocks_per_seq: int, seq_lens, n_slots: int) -> hsd_kv:
    return hsd_kv(k_pool.data_ptr(), v_pool.data_ptr(), n_blocks, block_table.data_ptr(), max_blocks_per_seq,
                  seq_lens.data_ptr(), n_slots)


def hsd_status_string(status: int) -> str:
    return _lib.hsd_status_string(status).decode()


def hsd_create(cfg: hsd_model_config, w: hsd_weights):
    """Returns (status, ctx handle)."""
    out = C.c_void_p()
    st = _lib.hsd_create(C.byref(cfg) if cfg is not None else None, C.byref(w) if w is not None else None,
                         C.byref(out))
    return st, out


def hsd_destroy(ctx) -> int:
    return _lib.hsd_destroy(ctx)


def hsd_workspace_bytes(ctx, max_total_q: int, max_seqs: int) -> int:
    return int(_lib.hsd_workspace_bytes(ctx, max_total_q, max_seqs))


def hsd_prefill(ctx, kv, n_seqs, cu_len, embeds, token_ids, seq_slots, total_rows, max_len, first_token, workspace,
                ws_bytes, stream) -> int:
    return _lib.hsd_prefill(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(cu_len), _p(embeds),
                            _p(token_ids), _p(seq_slots), total_rows, max_len, _p(first_token), _p(workspace),
                            ws_bytes, _p(stream))


def hsd_verify_regions(ctx, kv, n_seqs, cu_q, q_tokens, seq_slots, max_q_len, total_q, log_tau, accept_len,
                       emit_tokens, n_emit, row_argmax, row_zmax, row_zdraft, workspace, ws_bytes, stream) -> int:
    return _lib.hsd_verify_regions(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(cu_q), _p(q_tokens),
                                   _p(seq_slots), max_q_len, total_q, log_tau, _p(accept_len), _p(emit_tokens),
                                   _p(n_emit), _p(row_argmax), _p(row_zmax), _p(row_zdraft), _p(workspace), ws_bytes,
                                   _p(stream))


def hsd_verify_page(ctx, kv, seq_slot, pending_token, draft_chunk, chunk_len, log_tau, accept_len, emit_tokens,
                    n_emit, row_argmax, row_zmax, row_zdraft, workspace, ws_bytes, stream) -> int:
    return _lib.hsd_verify_page(ctx, C.byref(kv) if kv is not None else None, seq_slot, _p(pending_token),
                                _p(draft_chunk), chunk_len, log_tau, _p(accept_len), _p(emit_tokens), _p(n_emit),
                                _p(row_argmax), _p(row_zmax), _p(row_zdraft), _p(workspace), ws_bytes, _p(stream))


def hsd_verify_regions_host(ctx, kv, n_seqs, cu_q, q_tokens, seq_slots, log_tau, commit, accept_len, emit_tokens, n_emit,
                            workspace, ws_bytes, stream):
    """Host-buffer form: cu_q, q_tokens, accept_len, emit_tokens, n_emit are HOST tensors (CPU torch tensors or
    addresses).  Returns (status, max_q_len)."""
    mq = C.c_int(0)
    st = _lib.hsd_verify_regions_host(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(cu_q), _p(q_tokens),
                                      _p(seq_slots), log_tau, int(commit), _p(accept_len), _p(emit_tokens), _p(n_emit),
                                      C.byref(mq), _p(workspace), ws_bytes, _p(stream))
    return st, mq.value


def hsd_kv_commit(ctx, kv, n_seqs, seq_slots, accept_len, blocks_in_use, stream) -> int:
    return _lib.hsd_kv_commit(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(seq_slots), _p(accept_len),
                              _p(blocks_in_use), _p(stream))


def hsd_verify_tree(ctx, kv, n_seqs, cu_q, q_tokens, parent, seq_slots, max_q_len, total_q, log_tau, accept_len,
                    emit_tokens, n_emit, accept_rows, row_argmax, row_zmax, row_zchild, workspace, ws_bytes, stream) -> int:
    return _lib.hsd_verify_tree(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(cu_q), _p(q_tokens), _p(parent),
                                _p(seq_slots), max_q_len, total_q, log_tau, _p(accept_len), _p(emit_tokens), _p(n_emit),
                                _p(accept_rows), _p(row_argmax), _p(row_zmax), _p(row_zchild), _p(workspace), ws_bytes,
                                _p(stream))


def hsd_kv_commit_tree(ctx, kv, n_seqs, seq_slots, accept_len, accept_rows, max_q_len, blocks_in_use, stream) -> int:
    return _lib.hsd_kv_commit_tree(ctx, C.byref(kv) if kv is not None else None, n_seqs, _p(seq_slots), _p(accept_len),
                                   _p(accept_rows), max_q_len, _p(blocks_in_use), _p(stream))


def hsd_dsv_build(ctx, n_seqs, window_n, window, emit_tokens, n_emit, emit_stride, draft_tokens, total_draft_tokens,
                  draft_off, n_drafts, seq_draft_off, max_rows, q_tokens, parent, cu_q, n_rows, stream, seq_map=None,
                  n_owners: int = 0) -> int:
    return _lib.hsd_dsv_build(ctx, n_seqs, window_n, _p(window), _p(emit_tokens), _p(n_emit), emit_stride,
                              _p(draft_tokens), total_draft_tokens, _p(draft_off), n_drafts, _p(seq_draft_off), max_rows,
                              _p(q_tokens), _p(parent), _p(cu_q), _p(n_rows), _p(seq_map), n_owners, _p(stream))


def make_stage(n_lanes, n_seqs, window_n, out_stride, idle_slot, lane_seq, lane_slot, window, first_token, seq_slot,
               max_new, out_tokens, out_len, seq_steps, seq_accepted, counters) -> hsd_stage:
    ptr = lambda t: None if t is None else t.data_ptr()
    return hsd_stage(n_lanes, n_seqs, window_n, out_stride, idle_slot, ptr(lane_seq), ptr(lane_slot), ptr(window),
                     ptr(first_token), ptr(seq_slot), ptr(max_new), ptr(out_tokens), ptr(out_len), ptr(seq_steps),
                     ptr(seq_accepted), ptr(counters))


def hsd_stage_begin(ctx, stage, kv, stream) -> int:
    return _lib.hsd_stage_begin(ctx, C.byref(stage) if stage is not None else None,
                                C.byref(kv) if kv is not None else None, _p(stream))


def hsd_stage_advance(ctx, stage, kv, accept_len, emit_tokens, n_emit, emit_stride, stream) -> int:
    return _lib.hsd_stage_advance(ctx, C.byref(stage) if stage is not None else None,
                                  C.byref(kv) if kv is not None else None, _p(accept_len), _p(emit_tokens), _p(n_emit),
                                  emit_stride, _p(stream))


def hsd_stage_aggregate(ctx, stage, draft_tokens, capacity, draft_off, stream) -> int:
    return _lib.hsd_stage_aggregate(ctx, C.byref(stage) if stage is not None else None, _p(draft_tokens), capacity,
                                    _p(draft_off), _p(stream))


def hsd_device_status(ctx, workspace, stream):
    """Returns (status, [code, where, 0, 0])."""
    buf = (C.c_int * 4)()
    st = _lib.hsd_device_status(ctx, _p(workspace), _p(stream), buf)
    return st, list(buf)


def hsd_last_cuda_error(ctx) -> int:
    return _lib.hsd_last_cuda_error(ctx)


def hsd_launch_count(ctx) -> int:
    return int(_lib.hsd_launch_count(ctx))


def hsd_profile_enable(ctx, enable: int) -> int:
    return _lib.hsd_profile_enable(ctx, enable)


def hsd_profile_read(ctx):
    """Returns (status_or_count, {kernel class: (total_ms, launches)})."""
    cap = 32
    names = (C.c_char_p * cap)()
    ms = (C.c_double * cap)()
    n = (C.c_longlong * cap)()
    r = _lib.hsd_profile_read(ctx, cap, names, ms, n)
    out = {}
    for k in range(max(0, min(r, cap))):
        out[names[k].decode()] = (ms[k], int(n[k]))
    return r, out


def hsd_debug_logits(ctx, workspace, total_q, n_seqs, logits, stream) -> int:
    return _lib.hsd_debug_logits(ctx, _p(workspace), total_q, n_seqs, _p(logits), _p(stream))


def hsd_debug_buffer(ctx, workspace, total_q, n_seqs, name: str):
    """Returns (status, address, bytes)."""
    ptr, sz = C.c_void_p(), C.c_size_t()
    st = _lib.hsd_debug_buffer(ctx, _p(workspace), total_q, n_seqs, name.encode(), C.byref(ptr), C.byref(sz))
    return st, ptr.value, sz.value


def hsd_debug_tap(ctx, layer: int, which: int, dst, dst_bytes: int) -> int:
    """Arms a tap: the next forward copies intermediate `which` (HSD_TAP_*) of decoder layer `layer` into dst."""
    return _lib.hsd_debug_tap(ctx, layer, which, _p(dst), dst_bytes)


def hsd_debug_set_gemm_tile(ctx, tile_n: int, k_slices: int) -> int:
    return _lib.hsd_debug_set_gemm_tile(ctx, tile_n, k_slices)


def hsd_debug_set_attn_plan(ctx, target_items: int, min_kv_tiles: int) -> int:
    return _lib.hsd_debug_set_attn_plan(ctx, target_items, min_kv_tiles)


def hsd_op_linear(ctx, A, W, Cout, M, n_out, K, mode, stream) -> int:
    return _lib.hsd_op_linear(ctx, _p(A), _p(W), _p(Cout), M, n_out, K, mode, _p(stream))


def hsd_op_lm_head_argmax(ctx, h, rows, next_tokens, scratch, scratch_bytes, argmax, zmax, zdraft, stream) -> int:
    return _lib.hsd_op_lm_head_argmax(ctx, _p(h), rows, _p(next_tokens), _p(scratch), scratch_bytes, _p(argmax),
                                      _p(zmax), _p(zdraft), _p(stream))


def hsd_op_lm_head_argmax_noalloc(ctx, h, rows, next_tokens, argmax, zmax, zdraft, stream) -> int:
    """LM-head argmax for callers that cannot allocate: the scratch is a fixed array inside the library
    (at most HSD_NOALLOC_MAX_ROWS rows; calls that may overlap on the GPU race on it)."""
    return _lib.hsd_op_lm_head_argmax_noalloc(ctx, _p(h), rows, _p(next_tokens), _p(argmax), _p(zmax), _p(zdraft),
                                              _p(stream))
