"""CPU oracle for the two-stage decode loop of Hierarchical Speculative Decoding.

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's cpu-baseline / reference arm may
import this module; the CUDA library never does, and this module imports nothing from the CUDA path.  Plain Python
around the two other oracles (the decoder / acceptance oracle and the matching / packing oracle), not tuned.

What it computes (paper Sec. 3.1):
  * SpecDecode(p_theta, z, Y~) (Eq. 1): starting from the prefilled visual input z, repeat the decoupled-verification
    step of Sec. 3.2 — reference window over the accepted tokens, matching against the FIXED draft set (Eq. 5, 6),
    prefix tree (Eq. 7), one forward over the packed tree (Eq. 8), greedy traversal (Eq. 9-11), append pi(s) + u_hat
    (Eq. 12), keep the accepted rows' K/V and drop the rest (Sec. 4.2) — until the output has its length;
  * Stage 1 (Eq. 2): SpecDecode on every region crop with that region's drafts, independently;
  * the page draft (Eq. 3): the set of Stage-1 outputs, kept fixed;
  * Stage 2 (Eq. 4): SpecDecode on the full page with the page draft;
  * the step statistics of Sec. 4.2: verification steps N, accepted draft tokens alpha_k per step, AAL = mean alpha_k.

Readings where the paper is silent:
  * when an output ends: the paper's parsers stop at their end-of-sequence token; the synthetic decoders here have
    none, so every call gets a token budget `max_new` and stops at the first step that reaches it (the output is cut
    to the budget; the cut-off tokens of that last step are not counted as accepted);
  * the first token of an output is the prefill's greedy token (it is the pending token of the first step);
  * while fewer than n tokens have been accepted the window is not full, nothing matches, and the step is a plain
    one-token decode step (the packed tree is its root).

Pins (tests/test_two_stage_oracle.py): with tau = 1 the output equals plain greedy decoding whatever the drafts are
(speculation is lossless under exact-match acceptance); a draft equal to the model's own text is consumed 127 tokens
+ 1 bonus token per step, which fixes the step count in closed form; steps / tokens = 1 / (AAL + 1), the identity the
paper's printed numbers satisfy; Stage 2 receives exactly the Stage-1 outputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from . import dsv_oracle as D
from . import hsd_oracle as O


@dataclass
class DecodeTrace:
    tokens: List[int]                      # the verified output y_hat (first token = the prefill's greedy token)
    accepted_per_step: List[int] = field(default_factory=list)   # alpha_k of every verification step
    rows_per_step: List[int] = field(default_factory=list)       # packed rows (root + nodes) of every step
    token_gap: List[float] = field(default_factory=list)         # per output token: top-1 / top-2 logit gap of the row
                                                                 # that chose it (how clear-cut that decision was)

    @property
    def steps(self) -> int:
        return len(self.accepted_per_step)

    @property
    def aal(self) -> float:
        return float(np.mean(self.accepted_per_step)) if self.accepted_per_step else 0.0


def spec_decode(seq: O.CachedSequence, first_token: int, drafts: Sequence[Sequence[int]], max_new: int, n: int = 3,
                max_rows: int = 128, log_tau: float = 0.0, max_candidates: int = 64) -> DecodeTrace:
    """SpecDecode (Eq. 1) on a prefilled sequence: `first_token` is the prefill's greedy token (already part of the
    output, not yet in the cache).  Returns the output of `max_new` tokens and the per-step statistics."""
    out = [int(first_token)]
    trace = DecodeTrace(out)
    pl = np.sort(seq.last_prefill_logits)
    trace.token_gap.append(float(pl[-1] - pl[-2]))
    while len(out) < max_new:
        q_tokens, parent = D.pack(out, drafts, n, max_rows, max_candidates)        # window = last n accepted tokens
        res = O.verify_cached(seq, q_tokens[0], np.asarray(q_tokens[1:], np.int64), np.asarray(parent), log_tau)
        O.commit_step(seq, res)                                                     # pending row + accepted path stay
        room = max_new - len(out)
        out.extend(res.emitted[:room])
        trace.token_gap.extend(float(res.row_gap[node]) for node in ([0] + list(res.path))[:room])
        trace.accepted_per_step.append(min(res.accept_len, room))
        trace.rows_per_step.append(len(q_tokens))
    return trace


@dataclass
class RegionInput:
    prefix_embeds: Optional[np.ndarray]    # [L, d] rows used where prefix_ids < 0
    prefix_ids: np.ndarray                 # [L]
    drafts: List[List[int]]                # the pipeline's drafts for this region (fixed)
    max_new: int                           # output length of the region


@dataclass
class PageResult:
    region_traces: List[DecodeTrace]
    page_draft: List[List[int]]            # Eq. 3: the Stage-1 outputs
    page_trace: DecodeTrace

    def summary(self):
        s1 = [a for t in self.region_traces for a in t.accepted_per_step]
        s2 = self.page_trace.accepted_per_step
        return {"stage1_steps": len(s1), "stage1_tokens": sum(len(t.tokens) for t in self.region_traces),
                "stage1_aal": float(np.mean(s1)) if s1 else 0.0, "stage2_steps": len(s2),
                "stage2_tokens": len(self.page_trace.tokens), "stage2_aal": float(np.mean(s2)) if s2 else 0.0}


def hierarchical_decode(model: O.Decoder, regions: Sequence[RegionInput], page: RegionInput, n: int = 3,
                        max_rows: int = 128, log_tau: float = 0.0) -> PageResult:
    """The two-stage hierarchy of Sec. 3.1.  `page.drafts` is ignored: the page draft is the set of Stage-1 outputs."""
    traces = []
    for r in regions:                                   # Stage 1 (Eq. 2): regions are independent
        seq = O.CachedSequence(model)
        first = seq.prefill(r.prefix_embeds, r.prefix_ids)
        traces.append(spec_decode(seq, first, r.drafts, r.max_new, n, max_rows, log_tau))
    page_draft = [list(t.tokens) for t in traces]       # Eq. 3, kept fixed during Stage 2
    seq = O.CachedSequence(model)
    first = seq.prefill(page.prefix_embeds, page.prefix_ids)
    page_trace = spec_decode(seq, first, page_draft, page.max_new, n, max_rows, log_tau)    # Stage 2 (Eq. 4)
    return PageResult(traces, page_draft, page_trace)
