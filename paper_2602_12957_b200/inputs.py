"""Seeded synthetic inputs for the HSD draft-verification step.

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/bench.  It holds no arithmetic of the method: it draws random weights, visual
embedding rows, token ids, lengths and block tables from a fixed-seed generator and
packs them into plain numpy arrays.  Everything that needs the decoder (the greedy
continuation a draft agrees with, logits, acceptance) is passed in by the caller.

Workload shapes follow the five benchmark configurations (Tiny verify, Region-level
stage, Page-level stage, Long-document page verify, Mixed serving batch); they stand
in for the document-parsing benchmarks of the paper's Sec. 4.1, whose pages, target
VLM weights and pipeline drafter are not available offline.

Draw order inside one `numpy.random.Generator(PCG64(seed))` stream is fixed:
weights layer by layer -> (new stream) lengths -> visual rows -> token ids ->
agreement lengths -> random draft tokens -> block permutation.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

BASE_SEED = 12957


# --------------------------------------------------------------------------- config
@dataclass(frozen=True)
class ModelConfig:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-6
    kv_block: int = 64
    qk_norm: bool = False      # per-head RMSNorm of q and k before the rotary embedding (Qwen3-style decoders)

    @property
    def qkv_out(self) -> int:
        return (self.n_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def streamed_params(self) -> int:
        """Weights read once per forward (embedding table excluded: it is gathered)."""
        d, f = self.d_model, self.d_ffn
        per_layer = self.qkv_out * d + d * self.n_heads * self.head_dim + 2 * f * d + d * f + 2 * d
        return self.n_layers * per_layer + self.vocab * d + d

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * 2 * self.n_layers


TINY = ModelConfig(n_layers=1, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=1024, vocab=4096)
DECODER = ModelConfig(n_layers=24, d_model=1024, n_heads=16, n_kv_heads=8, head_dim=64, d_ffn=4096, vocab=32768)


def small_decoder(n_layers: int = 2, vocab: int = 8192) -> ModelConfig:
    """Same per-layer shape as the 24-layer decoder, fewer layers / smaller vocabulary,
    for parity cases the CPU oracle finishes in seconds."""
    return ModelConfig(n_layers=n_layers, d_model=1024, n_heads=16, n_kv_heads=8, head_dim=64,
                       d_ffn=4096, vocab=vocab)


# --------------------------------------------------------------------------- bf16 helpers
def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Values representable in bf16, widened back to float32.  Both the oracle and the
    CUDA path receive exactly these values, so only their arithmetic differs."""
    return from_bf16_bits(to_bf16_bits(a))


# --------------------------------------------------------------------------- weights
def make_weights(cfg: ModelConfig, seed: int) -> Dict[str, object]:
    """Random-init decoder weights, N(0, 0.02), gains 1 + 0.02 N(0,1), bf16-rounded float32.

    Linear weights are stored `[out_features, in_features]` (y = x @ W.T).
    `w_qkv` rows: q heads, then k heads, then v heads.  `w_gate_up` rows: gate then up.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    d, f, hd = cfg.d_model, cfg.d_ffn, cfg.head_dim

    def lin(o, i):
        return bf16_round(rng.standard_normal((o, i), dtype=np.float32) * np.float32(0.02))

    def gain():
        return bf16_round(np.float32(1.0) + np.float32(0.02) * rng.standard_normal(d, dtype=np.float32))

    layers = []
    for _ in range(cfg.n_layers):
        layers.append({
            "attn_norm": gain(),
            "w_qkv": lin(cfg.qkv_out, d),
            "w_o": lin(d, cfg.n_heads * hd),
            "ffn_norm": gain(),
            "w_gate_up": lin(2 * f, d),
            "w_down": lin(d, f),
        })
    out = {
        "layers": layers,
        "embed": lin(cfg.vocab, d),
        "final_norm": gain(),
        "lm_head": lin(cfg.vocab, d),
    }
    if cfg.qk_norm:     # drawn from a stream of their own, so every other weight is the same with and without them
        rq = np.random.Generator(np.random.PCG64(seed + 7_000_001))
        for lw in layers:
            for name in ("q_norm", "k_norm"):
                lw[name] = bf16_round(np.float32(1.0) + np.float32(0.1) * rq.standard_normal(hd, dtype=np.float32))
    return out


def make_chain_weights(cfg: ModelConfig, seed: int, branch_scale: float = 0.004):
    """Decoder weights whose greedy text is known in advance and decided by wide margins: (weights, order).

    `order` is a random cyclic order of the vocabulary; after token order[i] the decoder emits order[i + 1].  The
    weights are the random-init ones of `make_weights` except that the two projections that write into the residual
    stream (w_o, w_down) are scaled by `branch_scale`, so the last token's embedding row dominates the stream, and
    that the LM-head row of order[i + 1] is 4 x the embedding row of order[i] (the logit of the successor is the
    squared norm of an embedding row over its RMS, about 80; every other logit is a cross product, within +-12).
    Random-init weights have no such margins (half their rows have a top-1 / top-2 gap below 0.1), so a text decoded
    with them changes with the summation order of a kernel; loops whose statistics depend on WHICH tokens come out
    (accepted lengths over many steps) use these.  Every kernel runs the same dense arithmetic on them."""
    w = make_weights(cfg, seed)
    rng = np.random.Generator(np.random.PCG64(seed + 9_000_003))
    order = rng.permutation(cfg.vocab).astype(np.int64)
    for lw in w["layers"]:
        lw["w_o"] = bf16_round(lw["w_o"] * np.float32(branch_scale))
        lw["w_down"] = bf16_round(lw["w_down"] * np.float32(branch_scale))
    lm = np.empty_like(w["lm_head"])
    lm[np.roll(order, -1)] = w["embed"][order] * np.float32(4.0)       # exact in bf16
    w["lm_head"] = lm
    return w, order


# --------------------------------------------------------------------------- workloads
@dataclass
class SeqInput:
    """One sequence (a region crop or a page) before any decoder has seen it."""
    prefix_embeds: np.ndarray      # [L, d] float32 (bf16-rounded); rows used where prefix_ids < 0
    prefix_ids: np.ndarray         # [L] int32, -1 = visual row (use prefix_embeds), else token id
    draft_len: int                 # k
    agree_len: int                 # planted agreement length a in [0, k]
    rand_tokens: np.ndarray        # [k] int32 uniform tokens (mismatch + tail material)
    continue_on_greedy: bool       # page drafts: after the planted substitution follow the greedy path

    @property
    def prefix_len(self) -> int:
        return int(self.prefix_ids.shape[0])


@dataclass
class Workload:
    name: str
    cfg: ModelConfig
    seed: int
    seqs: List[SeqInput]
    chunk_len: Optional[int] = None      # page workloads: draft verified in chunks of this many tokens
    notes: str = ""


def lognormal_lengths(rng, n, mean, lo, hi, sigma=0.75):
    """k = clip(round(exp(N(mu, sigma^2))), lo, hi) with mu chosen so the unclipped mean is `mean`."""
    mu = np.log(mean) - 0.5 * sigma * sigma
    k = np.rint(np.exp(rng.normal(mu, sigma, size=n))).astype(np.int64)
    return np.clip(k, lo, hi).astype(np.int32)


def _visual_rows(rng, n, d):
    return bf16_round(rng.standard_normal((n, d), dtype=np.float32))


def _agree_mixture(rng, k, p_full, lo_frac):
    """a = k with probability p_full, else floor(U(lo_frac, 1) * k)."""
    full = rng.random() < p_full
    frac = rng.uniform(lo_frac, 1.0)
    return int(k) if full else int(np.floor(frac * k))


def tiny_workload(seed: int = BASE_SEED + 0, n_regions: int = 4, prefix_len: int = 128,
                  n_visual: int = 64, draft_len: int = 16, cfg: ModelConfig = TINY) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    seqs = []
    for _ in range(n_regions):
        emb = np.zeros((prefix_len, cfg.d_model), np.float32)
        emb[:n_visual] = _visual_rows(rng, n_visual, cfg.d_model)
        ids = np.full(prefix_len, -1, np.int32)
        ids[n_visual:] = rng.integers(0, cfg.vocab, size=prefix_len - n_visual, dtype=np.int32)
        a = int(rng.integers(0, draft_len + 1))
        seqs.append(SeqInput(emb, ids, draft_len, a,
                             rng.integers(0, cfg.vocab, size=draft_len, dtype=np.int32), False))
    return Workload("tiny", cfg, seed, seqs)


def region_workload(seed: int = BASE_SEED + 1, n_regions: int = 16, prefix_lo: int = 256, prefix_hi: int = 1024,
                    draft_mean: float = 64.0, draft_lo: int = 8, draft_hi: int = 256,
                    fixed_draft_len: Optional[int] = None, cfg: ModelConfig = DECODER,
                    name: str = "region") -> Workload:
    """Region-level stage: all-visual prefixes, lognormal draft lengths, mean acceptance 0.8."""
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    pl = rng.integers(prefix_lo, prefix_hi + 1, size=n_regions)
    if fixed_draft_len is None:
        ks = lognormal_lengths(rng, n_regions, draft_mean, draft_lo, draft_hi)
    else:
        ks = np.full(n_regions, fixed_draft_len, np.int32)
    seqs = []
    for i in range(n_regions):
        L, k = int(pl[i]), int(ks[i])
        emb = _visual_rows(rng, L, cfg.d_model)
        a = _agree_mixture(rng, k, 0.5, 0.2)
        seqs.append(SeqInput(emb, np.full(L, -1, np.int32), k, a,
                             rng.integers(0, cfg.vocab, size=k, dtype=np.int32), False))
    return Workload(name, cfg, seed, seqs)


def page_workload(seed: int = BASE_SEED + 2, n_visual: int = 4096, n_prompt: int = 256,
                  draft_len: int = 4096, chunk_len: int = 512, p_full: float = 0.75, lo_frac: float = 0.6,
                  cfg: ModelConfig = DECODER, name: str = "page") -> Workload:
    """Page-level stage: one sequence, visual rows then prompt token ids, a long refined draft
    verified chunk by chunk.  `agree_len` applies per chunk and is re-drawn by `page_chunk_agreement`."""
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    L = n_visual + n_prompt
    emb = np.zeros((L, cfg.d_model), np.float32)
    emb[:n_visual] = _visual_rows(rng, n_visual, cfg.d_model)
    ids = np.full(L, -1, np.int32)
    ids[n_visual:] = rng.integers(0, cfg.vocab, size=n_prompt, dtype=np.int32)
    a = _agree_mixture(rng, chunk_len, p_full, lo_frac)
    seq = SeqInput(emb, ids, draft_len, a, rng.integers(0, cfg.vocab, size=draft_len, dtype=np.int32), True)
    return Workload(name, cfg, seed, [seq], chunk_len=chunk_len)


def long_workload(seed: int = BASE_SEED + 3, chunk_len: int = 1024, cfg: ModelConfig = DECODER) -> Workload:
    return page_workload(seed=seed, n_visual=2048, n_prompt=0, draft_len=16384, chunk_len=chunk_len,
                         p_full=0.85, lo_frac=0.6, cfg=cfg, name=f"long{chunk_len}")


def mixed_workload(seed: int = BASE_SEED + 4, n_regions: int = 64, fixed_draft_len: Optional[int] = None,
                   with_page_chunks: bool = True, cfg: ModelConfig = DECODER) -> Workload:
    """Mixed serving batch: 64 regions (prefix U{128..2048}, lognormal drafts mean 96 clipped 8..512,
    per-region acceptance rate U(0.5,1)) plus two page-level chunks of 1024 tokens over 4352-token
    page prefixes, all in one varlen launch."""
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    pl = rng.integers(128, 2048 + 1, size=n_regions)
    ks = (lognormal_lengths(rng, n_regions, 96.0, 8, 512) if fixed_draft_len is None
          else np.full(n_regions, fixed_draft_len, np.int32))
    seqs = []
    for i in range(n_regions):
        L, k = int(pl[i]), int(ks[i])
        emb = _visual_rows(rng, L, cfg.d_model)
        a = int(np.floor(rng.uniform(0.5, 1.0) * k))
        seqs.append(SeqInput(emb, np.full(L, -1, np.int32), k, a,
                             rng.integers(0, cfg.vocab, size=k, dtype=np.int32), False))
    if with_page_chunks:
        for _ in range(2):
            L, k = 4352, 1024
            emb = _visual_rows(rng, L, cfg.d_model)
            a = _agree_mixture(rng, k, 0.75, 0.6)
            seqs.append(SeqInput(emb, np.full(L, -1, np.int32), k, a,
                                 rng.integers(0, cfg.vocab, size=k, dtype=np.int32), True))
    nm = "mixed" if fixed_draft_len is None else f"mixed_k{fixed_draft_len}"
    return Workload(nm, cfg, seed, seqs)


# --------------------------------------------------------------------------- drafts
def plant_draft(greedy: Sequence[int], k: int, agree_len: int, rand_tokens: np.ndarray, vocab: int,
                continue_on_greedy: bool) -> np.ndarray:
    """Build a k-token draft that copies `greedy` (some decoder's own greedy continuation, supplied by
    the caller) for `agree_len` tokens, then differs at that position.  Afterwards it is uniform-random
    (region drafts) or returns to the greedy path (page drafts: a substitution error, so the draft
    re-aligns right after the correction token)."""
    g = np.asarray(greedy, dtype=np.int64)
    a = int(min(agree_len, k))
    need = k if continue_on_greedy else min(a + 1, k)
    if g.shape[0] < need:
        raise ValueError(f"greedy continuation has {g.shape[0]} tokens, {need} needed")
    d = np.asarray(rand_tokens[:k], dtype=np.int64).copy()
    d[:a] = g[:a]
    if a < k:
        if d[a] == g[a]:
            d[a] = (d[a] + 1) % vocab
        if continue_on_greedy:
            d[a + 1:] = g[a + 1:k]
    return d.astype(np.int32)


# --------------------------------------------------------------------------- candidate trees
def plant_tree(greedy: Sequence[int], n_nodes: int, agree_len: int, vocab: int, seed: int, n_branches: int = 6,
               shuffle: bool = True):
    """A packed candidate tree of `n_nodes` nodes below the root (paper Sec. 3.2: suffixes merged on common
    prefixes).  One root-to-leaf "main" path copies `greedy` (some decoder's own greedy continuation, supplied by
    the caller) for `agree_len` tokens and then leaves it; `n_branches` side paths of random tokens fork off
    random nodes of the tree; siblings always carry distinct tokens, and a side branch never carries the greedy
    token of its depth, so the greedy path through the tree is unique.  Rows are packed parents-first but, with
    `shuffle`, otherwise in random order, so a row's index and its depth differ.

    Returns (tokens [n_nodes] int32 of rows 1.., parent [n_nodes + 1] int32 with parent[0] = -1, main_rows: the
    packed rows of the main path in depth order)."""
    rng = np.random.Generator(np.random.PCG64(seed + 3_000_017))
    g = [int(t) for t in greedy]
    n_nodes = int(n_nodes)
    if n_nodes < 1:
        return np.zeros(0, np.int32), np.asarray([-1], np.int32), []
    n_side = min(n_branches, max(0, n_nodes - 1))
    side_total = int(rng.integers(n_side, max(n_side, n_nodes // 2) + 1)) if n_side else 0
    main_len = n_nodes - side_total
    if len(g) < min(agree_len + 1, main_len):
        raise ValueError("greedy continuation too short for the planted agreement")
    # logical tree: node ids 1.., 0 = root
    par, tok, depth = [-1], [-1], [0]
    kids = {0: set()}

    def add(p, t):
        par.append(p); tok.append(int(t)); depth.append(depth[p] + 1)
        kids[p].add(int(t)); kids[len(par) - 1] = set()
        return len(par) - 1

    def fresh(p, avoid):
        while True:
            t = int(rng.integers(0, vocab))
            if t not in kids[p] and t != avoid:
                return t

    main, cur = [], 0
    a = int(min(agree_len, main_len))
    for d in range(main_len):
        gt = g[d] if d < len(g) else -1
        t = gt if d < a else fresh(cur, gt)
        cur = add(cur, t)
        main.append(cur)
    left = side_total
    for b in range(n_side):
        length = left if b == n_side - 1 else int(rng.integers(1, max(1, left - (n_side - 1 - b)) + 1))
        left -= length
        cur = int(rng.integers(0, len(par)))
        for _ in range(length):
            d = depth[cur]
            cur = add(cur, fresh(cur, g[d] if d < len(g) else -1))
    n = len(par)
    # packing order: random topological order (a node becomes available once its parent is placed)
    order, avail = [0], [j for j in range(1, n) if par[j] == 0]
    children = {j: [] for j in range(n)}
    for j in range(1, n):
        children[par[j]].append(j)
    while avail:
        pick = int(rng.integers(0, len(avail))) if shuffle else 0
        j = avail.pop(pick)
        order.append(j)
        avail.extend(children[j])
    where = {j: r for r, j in enumerate(order)}
    parent = np.asarray([-1] + [where[par[j]] for j in order[1:]], np.int32)
    tokens = np.asarray([tok[j] for j in order[1:]], np.int32)
    return tokens, parent, [where[j] for j in main]


# --------------------------------------------------------------------------- paged KV layout
def blocks_needed(n_tokens: int, kv_block: int = 64) -> int:
    return (int(n_tokens) + kv_block - 1) // kv_block


def make_block_tables(capacities: Sequence[int], seed: int, kv_block: int = 64, spare_blocks: int = 3):
    """Random physical placement: sequence i gets ceil(capacity_i / kv_block) distinct physical blocks drawn
    from a shuffled pool with a few unused blocks left over.  Returns (table [S, max_blocks] int32 padded
    with -1, n_physical_blocks)."""
    rng = np.random.Generator(np.random.PCG64(seed + 2_000_003))
    per = [blocks_needed(c, kv_block) for c in capacities]
    total = sum(per) + spare_blocks
    perm = rng.permutation(total).astype(np.int32)
    table = np.full((len(per), max(per) if per else 1), -1, np.int32)
    off = 0
    for i, n in enumerate(per):
        table[i, :n] = perm[off:off + n]
        off += n
    return table, total


def pack_queries(pending: Sequence[int], drafts: Sequence[np.ndarray]):
    """Packed query tokens [pending_i, d_i1..d_ik] for every sequence and the offsets cu_q [S+1]."""
    cu = [0]
    toks: List[int] = []
    for p, d in zip(pending, drafts):
        toks.append(int(p))
        toks.extend(int(t) for t in d)
        cu.append(len(toks))
    return np.asarray(toks, np.int32), np.asarray(cu, np.int32)
