"""Device-memory plumbing around the C-ABI calls: uploads weights, owns the paged KV pool, block table and
workspace as torch tensors, and marshals numpy inputs.  Every step of the method runs inside the library's
kernels; nothing here computes."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import inputs as I


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _bf16(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device=device, dtype=torch.bfloat16)


class DeviceModel:
    """Decoder weights on the device (bf16) plus the library context built over them."""

    def __init__(self, cfg: I.ModelConfig, weights: Dict[str, object], flags: int = 0, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("the HSD verify step needs a CUDA device (no CPU fallback)")
        self.cfg, self.device = cfg, torch.device(device)
        torch.cuda.set_device(self.device)
        up = lambda a: _bf16(a, self.device)
        self.embed, self.lm_head, self.final_norm = up(weights["embed"]), up(weights["lm_head"]), up(weights["final_norm"])
        self.layers = [{k: up(v) for k, v in lw.items()} for lw in weights["layers"]]
        self._cfg_c = B.make_config(cfg, flags)
        col = lambda k: [lw[k] for lw in self.layers]
        self._w_c = B.make_weights(self.embed, self.lm_head, self.final_norm, col("attn_norm"), col("w_qkv"), col("w_o"),
                                   col("ffn_norm"), col("w_gate_up"), col("w_down"),
                                   col("q_norm") if cfg.qk_norm else None, col("k_norm") if cfg.qk_norm else None)
        st, self.ctx = B.hsd_create(self._cfg_c, self._w_c)
        B.check(st, "hsd_create")

    def sibling(self, flags: int) -> "DeviceModel":
        """A second library context with other HSD_FLAG_* bits over the SAME device weights (nothing is copied)."""
        other = object.__new__(DeviceModel)
        other.cfg, other.device = self.cfg, self.device
        other.embed, other.lm_head, other.final_norm, other.layers = self.embed, self.lm_head, self.final_norm, self.layers
        other._cfg_c = B.make_config(self.cfg, flags)
        other._w_c = self._w_c
        st, other.ctx = B.hsd_create(other._cfg_c, other._w_c)
        B.check(st, "hsd_create")
        return other

    def close(self):
        if getattr(self, "ctx", None) is not None:
            B.hsd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class KvCache:
    """Caller-owned paged KV cache: pools, a block table with shuffled physical blocks, sequence lengths."""

    def __init__(self, model: DeviceModel, capacities: Sequence[int], seed: int = 0, poison: bool = False):
        cfg, dev = model.cfg, model.device
        table, n_blocks = I.make_block_tables(capacities, seed, cfg.kv_block)
        self.n_slots, self.n_blocks, self.max_blocks = len(capacities), n_blocks, table.shape[1]
        shape = (cfg.n_layers, n_blocks, cfg.n_kv_heads, cfg.kv_block, cfg.head_dim)
        if poison:   # huge finite filler: an unmasked read of a row that was never written wrecks the outputs
            self.k_pool = torch.full(shape, 1e30, dtype=torch.bfloat16, device=dev)
            self.v_pool = torch.full(shape, 1e30, dtype=torch.bfloat16, device=dev)
        else:
            self.k_pool = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
            self.v_pool = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
        self.table_host = table
        self.block_table = torch.from_numpy(np.where(table < 0, 0, table).astype(np.int32)).to(dev)
        self.seq_lens = torch.zeros(self.n_slots, dtype=torch.int32, device=dev)
        self.c = B.make_kv(self.k_pool, self.v_pool, n_blocks, self.block_table, self.max_blocks, self.seq_lens,
                           self.n_slots)

    def bytes(self) -> int:
        return 2 * self.k_pool.numel() * 2


class Workspace:
    def __init__(self, model: DeviceModel, max_total_q: int, max_seqs: int):
        self.max_total_q, self.max_seqs = max_total_q, max_seqs
        self.bytes = B.hsd_workspace_bytes(model.ctx, max_total_q, max_seqs)
        raw = torch.empty(self.bytes + 1024, dtype=torch.uint8, device=model.device)
        off = (-raw.data_ptr()) % 1024
        self._raw = raw
        self.ptr = raw.data_ptr() + off


class Engine:
    """One model + one KV cache + one workspace; methods mirror the C-ABI calls."""

    def __init__(self, model: DeviceModel, kv: KvCache, max_total_q: int, max_seqs: int):
        self.model, self.kv = model, kv
        self.ws = Workspace(model, max_total_q, max_seqs)
        self.dev = model.device

    # -- helpers -------------------------------------------------------------------------------
    def _i32(self, a) -> torch.Tensor:
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(self.dev)

    def device_status(self):
        return B.hsd_device_status(self.model.ctx, self.ws.ptr, _stream())

    def check_device(self, what: str = ""):
        st, words = self.device_status()
        if st != B.HSD_OK:
            raise B.HsdError(st, f"{what} device status {words}")

    # -- calls ---------------------------------------------------------------------------------
    def prefill(self, embeds: Sequence[Optional[np.ndarray]], ids: Sequence[np.ndarray],
                slots: Optional[Sequence[int]] = None) -> torch.Tensor:
        """Prefix rows of several sequences in one call.  Returns first_token (device int32 [S])."""
        lens = [len(x) for x in ids]
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        all_ids = np.concatenate(ids).astype(np.int32)
        d = self.model.cfg.d_model
        emb_t = None
        if any(e is not None for e in embeds):
            emb = np.concatenate([e if e is not None else np.zeros((n, d), np.float32) for e, n in zip(embeds, lens)])
            emb_t = _bf16(emb, self.dev)
        first = torch.empty(len(ids), dtype=torch.int32, device=self.dev)
        st = B.hsd_prefill(self.model.ctx, self.kv.c, len(ids), self._i32(cu), emb_t, self._i32(all_ids),
                           None if slots is None else self._i32(slots), int(cu[-1]), int(max(lens)), first,
                           self.ws.ptr, self.ws.bytes, _stream())
        B.check(st, "hsd_prefill")
        return first

    def alloc_outputs(self, n_seqs: int, max_q_len: int, total_q: int):
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=self.dev)
        return {"accept_len": i32(n_seqs), "emit_tokens": i32(n_seqs, max_q_len), "n_emit": i32(n_seqs),
                "row_argmax": i32(total_q), "row_zmax": torch.empty(total_q, dtype=torch.float32, device=self.dev),
                "row_zdraft": torch.empty(total_q, dtype=torch.float32, device=self.dev)}

    def verify_regions(self, q_tokens: torch.Tensor, cu_q: torch.Tensor, max_q_len: int, total_q: int,
                       out: Optional[dict] = None, slots: Optional[torch.Tensor] = None, log_tau: float = 0.0):
        n_seqs = cu_q.numel() - 1
        out = out or self.alloc_outputs(n_seqs, max_q_len, total_q)
        st = B.hsd_verify_regions(self.model.ctx, self.kv.c, n_seqs, cu_q, q_tokens, slots, max_q_len, total_q, log_tau,
                                  out["accept_len"], out["emit_tokens"], out["n_emit"], out["row_argmax"],
                                  out["row_zmax"], out["row_zdraft"], self.ws.ptr, self.ws.bytes, _stream())
        B.check(st, "hsd_verify_regions")
        return out

    def verify_tree(self, q_tokens: torch.Tensor, cu_q: torch.Tensor, parent: torch.Tensor, max_q_len: int,
                    total_q: int, out: Optional[dict] = None, slots: Optional[torch.Tensor] = None,
                    log_tau: float = 0.0):
        """Candidate trees (the workspace must have been sized for 2 * total_q rows)."""
        n_seqs = cu_q.numel() - 1
        if out is None:
            out = self.alloc_outputs(n_seqs, max_q_len, total_q)
            out["accept_rows"] = torch.zeros(n_seqs, max_q_len, dtype=torch.int32, device=self.dev)
            out["row_zchild"] = out.pop("row_zdraft")
        st = B.hsd_verify_tree(self.model.ctx, self.kv.c, n_seqs, cu_q, q_tokens, parent, slots, max_q_len, total_q,
                               log_tau, out["accept_len"], out["emit_tokens"], out["n_emit"], out["accept_rows"],
                               out["row_argmax"], out["row_zmax"], out["row_zchild"], self.ws.ptr, self.ws.bytes,
                               _stream())
        B.check(st, "hsd_verify_tree")
        return out

    def dsv_build(self, window: torch.Tensor, draft_tokens: torch.Tensor, draft_off: torch.Tensor,
                  seq_draft_off: torch.Tensor, max_rows: int, emit_tokens: Optional[torch.Tensor] = None,
                  n_emit: Optional[torch.Tensor] = None, out: Optional[dict] = None,
                  seq_map: Optional[torch.Tensor] = None):
        """Matching + prefix-tree packing on the device; `window` [S, n] is updated in place.  With `seq_map` [S]
        sequence i uses the drafts of owner seq_map[i] of `seq_draft_off` (lane batches)."""
        S, n = int(window.shape[0]), int(window.shape[1])
        if out is None:
            i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=self.dev)
            out = {"q_tokens": i32(S * max_rows), "parent": i32(S * max_rows), "cu_q": i32(S + 1), "n_rows": i32(S)}
        st = B.hsd_dsv_build(self.model.ctx, S, n, window, emit_tokens, n_emit,
                             int(emit_tokens.shape[1]) if emit_tokens is not None else 0, draft_tokens,
                             int(draft_tokens.numel()), draft_off, int(draft_off.numel()) - 1, seq_draft_off, max_rows,
                             out["q_tokens"], out["parent"], out["cu_q"], out["n_rows"], _stream(), seq_map,
                             int(seq_draft_off.numel()) - 1)
        B.check(st, "hsd_dsv_build")
        return out

    def commit_tree(self, accept_len: torch.Tensor, accept_rows: torch.Tensor, slots: Optional[torch.Tensor] = None,
                    blocks_in_use: Optional[torch.Tensor] = None):
        st = B.hsd_kv_commit_tree(self.model.ctx, self.kv.c, int(accept_len.numel()), slots, accept_len, accept_rows,
                                  int(accept_rows.shape[1]), blocks_in_use, _stream())
        B.check(st, "hsd_kv_commit_tree")

    def verify_page(self, slot: int, pending: torch.Tensor, chunk: torch.Tensor, out: Optional[dict] = None,
                    log_tau: float = 0.0):
        n = int(chunk.numel())
        out = out or self.alloc_outputs(1, n + 1, n + 1)
        st = B.hsd_verify_page(self.model.ctx, self.kv.c, slot, pending, chunk if n else None, n, log_tau,
                               out["accept_len"], out["emit_tokens"], out["n_emit"], out["row_argmax"], out["row_zmax"],
                               out["row_zdraft"], self.ws.ptr, self.ws.bytes, _stream())
        B.check(st, "hsd_verify_page")
        return out

    def commit(self, accept_len: torch.Tensor, slots: Optional[torch.Tensor] = None,
               blocks_in_use: Optional[torch.Tensor] = None):
        st = B.hsd_kv_commit(self.model.ctx, self.kv.c, int(accept_len.numel()), slots, accept_len, blocks_in_use,
                             _stream())
        B.check(st, "hsd_kv_commit")

    def debug_logits(self, total_q: int, n_seqs: int) -> torch.Tensor:
        z = torch.empty(total_q, self.model.cfg.vocab, dtype=torch.float32, device=self.dev)
        B.check(B.hsd_debug_logits(self.model.ctx, self.ws.ptr, total_q, n_seqs, z, _stream()), "hsd_debug_logits")
        return z
