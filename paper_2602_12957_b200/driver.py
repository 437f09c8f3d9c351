"""Two-stage decode loop (paper Sec. 3.1) over the C-ABI calls: Stage 1 runs the decoupled-verification step on a lane
batch of regions until every region's output is complete, finished regions making room for waiting ones; the outputs
become the page draft (Eq. 3); Stage 2 runs the same loop on the full page with one lane.

Everything that decides anything runs in the library's kernels: matching and tree packing (hsd_dsv_build), the forward
and the traversal (hsd_verify_tree), KV compaction and commit (hsd_kv_commit_tree), output bookkeeping, retirement and
lane hand-over (hsd_stage_advance), aggregation (hsd_stage_aggregate).  This module owns tensors, captures a few steps
into a CUDA graph and polls one counter to know when a stage is over."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import runtime as R


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


@dataclass
class StageResult:
    tokens: List[np.ndarray]         # output of every sequence
    steps: np.ndarray                # verification steps spent on every sequence
    accepted: np.ndarray             # accepted draft tokens of every sequence
    batch_steps: int                 # steps the lane batch took
    ms: float                        # device time of the loop

    @property
    def aal(self) -> float:
        return float(self.accepted.sum()) / max(1, int(self.steps.sum()))


class LaneBatch:
    """A lane batch over sequences that are already prefilled into KV slots 0 .. n_seqs-1 of `eng.kv` (the slot after
    them, n_seqs, is the idle slot)."""

    def __init__(self, eng: R.Engine, first_token: torch.Tensor, max_new: Sequence[int], draft_tokens: torch.Tensor,
                 draft_off: torch.Tensor, seq_draft_off: torch.Tensor, n_lanes: int, window_n: int = 3,
                 max_rows: int = 128, log_tau: float = 0.0):
        self.eng, dev = eng, eng.dev
        self.n_seqs, self.n_lanes = int(first_token.numel()), int(n_lanes)
        self.window_n, self.max_rows, self.log_tau = window_n, max_rows, float(log_tau)
        i32 = lambda *shape: torch.zeros(*shape, dtype=torch.int32, device=dev)
        self.out_stride = int(max(max_new)) + 1
        self.first_token = first_token
        self.max_new = eng._i32(np.asarray(max_new, np.int32))
        self.lane_seq, self.lane_slot = i32(self.n_lanes), i32(self.n_lanes)
        self.window = i32(self.n_lanes, window_n)
        self.out_tokens, self.out_len = i32(self.n_seqs, self.out_stride), i32(self.n_seqs)
        self.seq_steps, self.seq_accepted, self.counters = i32(self.n_seqs), i32(self.n_seqs), i32(4)
        self.stage = B.make_stage(self.n_lanes, self.n_seqs, window_n, self.out_stride, self.n_seqs, self.lane_seq,
                                  self.lane_slot, self.window, self.first_token, None, self.max_new, self.out_tokens,
                                  self.out_len, self.seq_steps, self.seq_accepted, self.counters)
        self.draft_tokens, self.draft_off, self.seq_draft_off = draft_tokens, draft_off, seq_draft_off
        T = self.n_lanes * max_rows
        self.build_out = {"q_tokens": i32(T), "parent": i32(T), "cu_q": i32(self.n_lanes + 1), "n_rows": i32(self.n_lanes)}
        self.out = eng.alloc_outputs(self.n_lanes, max_rows, T)
        self.out["accept_rows"] = i32(self.n_lanes, max_rows)
        self.out["row_zchild"] = self.out.pop("row_zdraft")
        self.graph = None

    def begin(self):
        B.check(B.hsd_stage_begin(self.eng.model.ctx, self.stage, self.eng.kv.c, _stream()), "hsd_stage_begin")

    def step(self):
        eng, o = self.eng, self.out
        eng.dsv_build(self.window, self.draft_tokens, self.draft_off, self.seq_draft_off, self.max_rows,
                      out=self.build_out, seq_map=self.lane_seq)
        eng.verify_tree(self.build_out["q_tokens"], self.build_out["cu_q"], self.build_out["parent"], self.max_rows,
                        self.n_lanes * self.max_rows, out=o, slots=self.lane_slot, log_tau=self.log_tau)
        eng.commit_tree(o["accept_len"], o["accept_rows"], slots=self.lane_slot)
        B.check(B.hsd_stage_advance(eng.model.ctx, self.stage, eng.kv.c, o["accept_len"], o["emit_tokens"], o["n_emit"],
                                    self.max_rows, _stream()), "hsd_stage_advance")

    def run(self, steps_per_poll: int = 8, use_graph: bool = True, max_polls: int = 100000) -> StageResult:
        """Steps until every sequence has its length.  `steps_per_poll` steps run back to back (one CUDA graph) between
        two reads of the "sequences not finished" counter; steps past the end only spin idle lanes."""
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.begin()
        self.step()                                   # eager once: sets the one-time kernel attributes before capture
        if use_graph and self.graph is None:
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph):      # (captures on a side stream; the calls below follow the current stream)
                for _ in range(steps_per_poll):
                    self.step()
        self.begin()                                  # restart cleanly after the trial step
        self.eng.kv.seq_lens.copy_(self._lens0)
        e0.record(stream)
        for _ in range(max_polls):
            if self.graph is not None:
                self.graph.replay()
            else:
                for _ in range(steps_per_poll):
                    self.step()
            if int(self.counters[1].item()) == 0:     # the one host read per poll
                break
        e1.record(stream)
        stream.synchronize()
        self.eng.check_device("lane batch")
        lens = self.out_len.cpu().numpy()
        toks = self.out_tokens.cpu().numpy()
        return StageResult([toks[r, :lens[r]].copy() for r in range(self.n_seqs)], self.seq_steps.cpu().numpy(),
                           self.seq_accepted.cpu().numpy(), int(self.counters[2].item()), e0.elapsed_time(e1))

    def remember_lengths(self):
        self._lens0 = self.eng.kv.seq_lens.clone()


@dataclass
class PageRun:
    stage1: StageResult
    stage2: StageResult
    prefill_ms: float
    aggregate_ms: float
    page_draft: List[np.ndarray]     # Eq. 3 as the device assembled it: one array per region


def run_page(model: R.DeviceModel, regions, region_drafts, region_max_new, page, page_max_new, n_lanes: int = 16,
             window_n: int = 3, max_rows: int = 128, log_tau: float = 0.0, steps_per_poll: int = 8,
             use_graph: bool = True, seed: int = 0, poison: bool = False,
             stage2_draft: Optional[Sequence[np.ndarray]] = None) -> PageRun:
    """The whole hierarchy for one page.  regions / page: (prefix_embeds [L, d] or None, prefix_ids [L]) pairs;
    region_drafts[i]: list of int arrays (the pipeline's drafts of region i); *_max_new: output lengths.
    `stage2_draft` (benchmarks with synthetic decoders only): drafts Stage 2 matches against INSTEAD of the aggregated
    Stage-1 outputs, which are still assembled and returned."""
    dev = model.device
    stream = torch.cuda.current_stream()
    n_reg = len(regions)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    # ---- prefill of all region crops (one call) and of the page (one call): support work, timed on its own
    caps = [len(ids) + m + 2 * max_rows + 2 for (_, ids), m in zip(regions, region_max_new)] + [2 * max_rows]
    kv1 = R.KvCache(model, caps, seed=seed, poison=poison)
    T1 = n_lanes * max_rows
    eng1 = R.Engine(model, kv1, max(sum(len(ids) for _, ids in regions), 2 * T1), max(n_reg + 1, n_lanes))
    kv2 = R.KvCache(model, [len(page[1]) + page_max_new + 2 * max_rows + 2, 2 * max_rows], seed=seed + 1, poison=poison)
    eng2 = R.Engine(model, kv2, max(len(page[1]), 2 * max_rows), 2)
    ev[0].record(stream)
    first1 = eng1.prefill([e for e, _ in regions], [i for _, i in regions], slots=list(range(n_reg)))
    first2 = eng2.prefill([page[0]], [page[1]], slots=[0])
    ev[1].record(stream)
    eng1.check_device("region prefill")
    eng2.check_device("page prefill")
    # ---- Stage 1: the pipeline's drafts, flattened
    toks, off, soff = [], [0], [0]
    for drafts in region_drafts:
        for d in drafts:
            toks.extend(int(t) for t in d)
            off.append(len(toks))
        soff.append(len(off) - 1)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    lb1 = LaneBatch(eng1, first1, region_max_new, i32(toks if toks else [0]), i32(off), i32(soff), n_lanes, window_n,
                    max_rows, log_tau)
    lb1.remember_lengths()
    s1 = lb1.run(steps_per_poll, use_graph)
    # ---- the page draft (Eq. 3) and Stage 2
    cap = int(sum(region_max_new)) + 1
    page_draft = torch.zeros(cap, dtype=torch.int32, device=dev)
    page_off = torch.zeros(n_reg + 1, dtype=torch.int32, device=dev)
    ev[2].record(stream)
    B.check(B.hsd_stage_aggregate(model.ctx, lb1.stage, page_draft, cap, page_off, _stream()), "hsd_stage_aggregate")
    ev[3].record(stream)
    d2_tok, d2_off, d2_n = page_draft, page_off, n_reg
    if stage2_draft is not None:
        flat, offs = [], [0]
        for d in stage2_draft:
            flat.extend(int(t) for t in d)
            offs.append(len(flat))
        d2_tok, d2_off, d2_n = i32(flat if flat else [0]), i32(offs), len(stage2_draft)
    lb2 = LaneBatch(eng2, first2, [page_max_new], d2_tok, d2_off, i32([0, d2_n]), 1, window_n, max_rows, log_tau)
    lb2.remember_lengths()
    s2 = lb2.run(steps_per_poll, use_graph)
    stream.synchronize()
    po, pd = page_off.cpu().numpy(), page_draft.cpu().numpy()
    return PageRun(s1, s2, ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3]),
                   [pd[po[r]:po[r + 1]].copy() for r in range(n_reg)])
