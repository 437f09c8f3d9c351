"""CPU oracle for one draft-verification step of Hierarchical Speculative Decoding.

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's
cpu-baseline / reference arm may import this module; the CUDA library never does, and
this module imports nothing from the CUDA path.  It is a plain, slow numpy restatement
of what the step computes; it is not tuned.

What it computes (paper Sec. 3.2, "Verification and acceptance"):
  * the target decoder's next-token scores for every node of a packed candidate
    sequence, each node conditioned on the accepted tokens plus its own ancestor path
    (Eq. 8; tree-ancestry mask of Fig. 2(c)); a linear draft is the chain-shaped tree;
  * the full-vocabulary argmax u_hat at each node (Eq. 10), the best admissible child
    u* (Eq. 9), the log-probability-gap acceptance test against log(tau) (Eq. 11);
  * the greedy traversal, its stop rules, and the emitted sequence pi(s) + u_hat (Eq. 12).

The decoder itself (pre-norm RMSNorm, rotary positions with rotate-half pairing,
grouped-query causal attention softmax(QK^T/sqrt(d))V, SwiGLU FFN, untied LM head, no
biases) is fixed by the benchmark configurations, not by the paper; `qk_norm` adds the per-head RMSNorm of q and k
before the rotary embedding that the Qwen3-family decoders the paper evaluates carry.

Readings where the paper is silent:
  * the most recent emitted token has no K/V yet ("pending" token); it is query row 0
    of the next step, so a k-token draft is k+1 query rows and full acceptance emits
    k+1 tokens (k draft tokens + the bonus token);
  * ties in an argmax go to the lowest token id; with tau = 1 acceptance is exact match
    with that argmax (Eq. 11 with a unique maximum);
  * log p(a) - log p(b) = z_a - z_b, so Eq. 11 is evaluated on raw logits.

Precision: float64 by default (`dtype=np.float32` is available for large cases); the
weights are whatever the caller supplies (the tests supply bf16-representable values).

Pins (tests/test_oracle_*.py): Hugging Face's Llama decoder as a library routine for the
whole forward; torch's scaled_dot_product_attention / rms_norm / silu; closed forms for
RoPE, RMSNorm and uniform-key attention; one verify call == k+1 single-token steps;
brute-force enumeration of all drafts on a tiny vocabulary against a literal tree walk;
the step-count identity the paper's printed numbers satisfy; the input rows (token rows
from the table, visual rows from the caller, id 0 a token) against the library decoder's
own embedding module fed with input_ids.  No function is unpinned.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------- pieces
def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing: dims (i, i + D/2) rotate by pos * base^(-2i/D).
    x: [T, H, D]; pos: [T]."""
    D = x.shape[-1]
    half = D // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / D)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]           # [T, half]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    e = s - np.max(s, axis=-1, keepdims=True)
    np.exp(e, out=e)
    e /= np.sum(e, axis=-1, keepdims=True)
    return e


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(D) + mask) v with grouped-query heads.
    q: [Tq, Hq, D]; k, v: [Tk, Hkv, D]; allowed: [Tq, Tk] bool (True = may attend).
    Query head g reads kv head g // (Hq / Hkv)."""
    Tq, Hq, D = q.shape
    group = Hq // k.shape[1]
    out = np.empty_like(q)
    neg = np.where(allowed, 0.0, -np.inf).astype(q.dtype)
    scale = 1.0 / math.sqrt(D)
    for g in range(Hq):
        kh = g // group
        s = q[:, g, :] @ k[:, kh, :].T
        s *= scale          # in place: the score matrix of a long context is large
        s += neg
        out[:, g, :] = softmax_rows(s) @ v[:, kh, :]
    return out


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def swiglu_ffn(h: np.ndarray, w_gate_up: np.ndarray, w_down: np.ndarray) -> np.ndarray:
    f = w_gate_up.shape[0] // 2
    gu = h @ w_gate_up.T
    return (silu(gu[:, :f]) * gu[:, f:]) @ w_down.T


# ----------------------------------------------------------------------------- model
@dataclass
class Decoder:
    """cfg: any object with n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab,
    rope_base, rms_eps.  weights: dict as produced by the seeded generator (float32 arrays,
    linear weights [out, in])."""
    cfg: object
    weights: Dict[str, object]
    dtype: type = np.float64

    def w(self, a: np.ndarray) -> np.ndarray:
        return a.astype(self.dtype, copy=False)

    def embed_rows(self, embeds: Optional[np.ndarray], ids: np.ndarray) -> np.ndarray:
        """Input rows: token id -> embedding-table row; id < 0 -> the given (visual) row."""
        ids = np.asarray(ids)
        x = self.w(self.weights["embed"][np.maximum(ids, 0)])
        if embeds is not None:
            x = np.where((ids < 0)[:, None], self.w(np.asarray(embeds)), x)
        elif np.any(ids < 0):
            raise ValueError("negative id without an embedding row")
        return np.ascontiguousarray(x)

    def logits(self, x_rows: np.ndarray) -> np.ndarray:
        h = rmsnorm(x_rows, self.w(self.weights["final_norm"]), self.cfg.rms_eps)
        return h @ self.w(self.weights["lm_head"]).T


def causal_allowed(n: int) -> np.ndarray:
    return np.tril(np.ones((n, n), dtype=bool))


def decoder_forward(model: Decoder, x: np.ndarray, pos: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    """Stateless forward of one sequence over ALL its rows (the ground truth, 'O-full').
    x: [n, d] input rows; pos: [n] rotary positions; allowed: [n, n] attention mask.
    Returns the residual stream after the last layer, [n, d]."""
    c = model.cfg
    Hq, Hkv, D = c.n_heads, c.n_kv_heads, c.head_dim
    x = x.astype(model.dtype, copy=True)
    for lw in model.weights["layers"]:
        h = rmsnorm(x, model.w(lw["attn_norm"]), c.rms_eps)
        qkv = h @ model.w(lw["w_qkv"]).T
        q = qkv[:, :Hq * D].reshape(-1, Hq, D)
        k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(-1, Hkv, D)
        v = qkv[:, (Hq + Hkv) * D:].reshape(-1, Hkv, D)
        if c.qk_norm:       # per-head RMSNorm over head_dim, before the rotary embedding
            q, k = rmsnorm(q, model.w(lw["q_norm"]), c.rms_eps), rmsnorm(k, model.w(lw["k_norm"]), c.rms_eps)
        q, k = rope(q, pos, c.rope_base), rope(k, pos, c.rope_base)
        o = attention(q, k, v, allowed).reshape(-1, Hq * D)
        x = x + o @ model.w(lw["w_o"]).T
        h = rmsnorm(x, model.w(lw["ffn_norm"]), c.rms_eps)
        x = x + swiglu_ffn(h, model.w(lw["w_gate_up"]), model.w(lw["w_down"]))
    return x


# ----------------------------------------------------------------------------- cached form
class CachedSequence:
    """'O-cached': contiguous per-layer K/V of the committed rows of one sequence."""

    def __init__(self, model: Decoder):
        c = model.cfg
        self.model = model
        self.k = [np.zeros((0, c.n_kv_heads, c.head_dim), model.dtype) for _ in range(c.n_layers)]
        self.v = [np.zeros((0, c.n_kv_heads, c.head_dim), model.dtype) for _ in range(c.n_layers)]
        self._spec = None          # (k_new, v_new) per layer of the last uncommitted call

    @property
    def length(self) -> int:
        return int(self.k[0].shape[0])

    def forward_rows(self, x_new: np.ndarray, depth: np.ndarray, allowed_new: np.ndarray) -> np.ndarray:
        """Run m new rows on top of the cache.  Row j sits at position length + depth[j], attends to
        every cached row and to new row i iff allowed_new[j, i].  The new rows' K/V are held as
        speculative until `commit`.  Returns the final residual rows [m, d]."""
        model, c = self.model, self.model.cfg
        Hq, Hkv, D = c.n_heads, c.n_kv_heads, c.head_dim
        L, m = self.length, x_new.shape[0]
        pos = L + np.asarray(depth, dtype=np.int64)
        allowed = np.concatenate([np.ones((m, L), dtype=bool), np.asarray(allowed_new, dtype=bool)], axis=1)
        x = x_new.astype(model.dtype, copy=True)
        spec = []
        for li, lw in enumerate(model.weights["layers"]):
            h = rmsnorm(x, model.w(lw["attn_norm"]), c.rms_eps)
            qkv = h @ model.w(lw["w_qkv"]).T
            q = qkv[:, :Hq * D].reshape(m, Hq, D)
            k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(m, Hkv, D)
            if c.qk_norm:
                q, k = rmsnorm(q, model.w(lw["q_norm"]), c.rms_eps), rmsnorm(k, model.w(lw["k_norm"]), c.rms_eps)
            q, k = rope(q, pos, c.rope_base), rope(k, pos, c.rope_base)
            v = qkv[:, (Hq + Hkv) * D:].reshape(m, Hkv, D)
            spec.append((k, v))
            o = attention(q, np.concatenate([self.k[li], k]), np.concatenate([self.v[li], v]), allowed)
            x = x + o.reshape(m, Hq * D) @ model.w(lw["w_o"]).T
            h = rmsnorm(x, model.w(lw["ffn_norm"]), c.rms_eps)
            x = x + swiglu_ffn(h, model.w(lw["w_gate_up"]), model.w(lw["w_down"]))
        self._spec = spec
        return x

    def commit(self, keep_rows: Sequence[int]) -> None:
        """Append the listed speculative rows (in order) to the cache; all others are rolled back."""
        idx = np.asarray(list(keep_rows), dtype=np.int64)
        for li, (k, v) in enumerate(self._spec):
            self.k[li] = np.concatenate([self.k[li], k[idx]])
            self.v[li] = np.concatenate([self.v[li], v[idx]])
        self._spec = None

    def prefill(self, embeds: Optional[np.ndarray], ids: np.ndarray, chunk: int = 1024) -> int:
        """Run prefix rows through the decoder, keep all their K/V, return the greedy next token
        (the first pending token)."""
        ids = np.asarray(ids)
        last = None
        for s in range(0, ids.shape[0], chunk):
            e = None if embeds is None else embeds[s:s + chunk]
            x = self.model.embed_rows(e, ids[s:s + chunk])
            n = x.shape[0]
            out = self.forward_rows(x, np.arange(n), causal_allowed(n))
            self.commit(range(n))
            last = out[-1:]
        self.last_prefill_logits = self.model.logits(last)[0]
        return int(np.argmax(self.last_prefill_logits))


# ----------------------------------------------------------------------------- tree + acceptance
def chain_parents(k: int) -> np.ndarray:
    """Parent pointers of a linear draft: row 0 is the root (the pending token), node j's parent is j-1."""
    return np.arange(-1, k, dtype=np.int64)


def tree_depth_and_mask(parent: np.ndarray):
    """From parent pointers (parent[0] = -1, parent[j] < j) give each node's depth and the tree-ancestry
    mask: node j may attend to node i iff i is j or an ancestor of j (Sec. 3.2, Fig. 2(c))."""
    n = len(parent)
    depth = np.zeros(n, dtype=np.int64)
    allowed = np.zeros((n, n), dtype=bool)
    for j in range(n):
        allowed[j, j] = True
        p = int(parent[j])
        if j == 0:
            if p != -1:
                raise ValueError("row 0 must be the root")
            continue
        if not (0 <= p < j):
            raise ValueError("parent pointers must point to an earlier row")
        depth[j] = depth[p] + 1
        allowed[j] |= allowed[p]
    return depth, allowed


def greedy_traverse(logits: np.ndarray, tokens: np.ndarray, parent: np.ndarray, log_tau: float = 0.0):
    """Greedy traversal of the candidate tree (Eq. 9-12).

    logits[j] are the scores of the distribution at node j (row 0 = root).  tokens[j] (j >= 1) is
    the token node j carries.  At the current node s: Next(s) = tokens of s's children; u* = the child
    token with the highest score (Eq. 9); u_hat = full-vocabulary argmax, lowest id on ties (Eq. 10);
    move to child(s, u*) iff z[u*] - z[u_hat] >= log_tau (Eq. 11); stop if the test fails or s has no
    child.  Returns (path rows after the root, emitted tokens = pi(s) + [u_hat]) (Eq. 12)."""
    n = len(parent)
    children: List[List[int]] = [[] for _ in range(n)]
    for j in range(1, n):
        children[int(parent[j])].append(j)
    s, path = 0, []
    while True:
        z = logits[s]
        u_hat = int(np.argmax(z))                     # numpy returns the first (lowest) index on ties
        if not children[s]:
            break
        best = max(children[s], key=lambda j: (z[int(tokens[j])], -int(tokens[j])))
        if log_tau == 0.0:
            ok = int(tokens[best]) == u_hat           # tau = 1: exact match with the lowest-id argmax
        else:
            ok = (z[int(tokens[best])] - z[u_hat]) >= log_tau
        if not ok:
            break
        path.append(best)
        s = best
    emitted = [int(tokens[j]) for j in path] + [u_hat]
    return path, emitted


@dataclass
class VerifyResult:
    accept_len: int                 # number of accepted draft tokens (alpha of the AAL definition)
    emitted: List[int]              # accepted tokens + correction/bonus token
    path: List[int]                 # accepted rows (after the root)
    row_argmax: np.ndarray          # [k+1] u_hat per row
    row_zmax: np.ndarray            # [k+1] max logit per row
    row_zdraft: np.ndarray          # [k+1] logit of the next draft token (chains; NaN on the last row)
    row_gap: np.ndarray             # [k+1] top-1 minus top-2 logit
    logits: Optional[np.ndarray] = None


def _row_stats(logits: np.ndarray, next_tok: Optional[np.ndarray]):
    am = np.argmax(logits, axis=1)
    top2 = np.partition(logits, -2, axis=1)[:, -2:]
    zmax = top2[:, 1]
    gap = top2[:, 1] - top2[:, 0]
    zd = np.full(logits.shape[0], np.nan)
    if next_tok is not None:
        m = len(next_tok)
        zd[:m] = logits[np.arange(m), next_tok]
    return am, zmax, zd, gap


def verify_full(model: Decoder, prefix_embeds: Optional[np.ndarray], prefix_ids: np.ndarray, pending: int,
                draft: np.ndarray, parent: Optional[np.ndarray] = None, log_tau: float = 0.0,
                keep_logits: bool = False) -> VerifyResult:
    """One verification step, stateless: recompute the forward over prefix + [pending, candidates]."""
    draft = np.asarray(draft, dtype=np.int64)
    k = len(draft)
    parent = chain_parents(k) if parent is None else np.asarray(parent)
    depth, allowed_new = tree_depth_and_mask(parent)
    L = len(prefix_ids)
    ids = np.concatenate([np.asarray(prefix_ids, dtype=np.int64), [pending], draft])
    emb = None
    if prefix_embeds is not None:
        emb = np.concatenate([prefix_embeds, np.zeros((k + 1, prefix_embeds.shape[1]), prefix_embeds.dtype)])
    x = model.embed_rows(emb, ids)
    n = L + k + 1
    allowed = np.zeros((n, n), dtype=bool)
    allowed[:L, :L] = causal_allowed(L)
    allowed[L:, :L] = True
    allowed[L:, L:] = allowed_new
    pos = np.concatenate([np.arange(L), L + depth])
    out = decoder_forward(model, x, pos, allowed)
    z = model.logits(out[L:])
    return _finish(z, draft, parent, log_tau, keep_logits)


def verify_cached(seq: CachedSequence, pending: int, draft: np.ndarray, parent: Optional[np.ndarray] = None,
                  log_tau: float = 0.0, keep_logits: bool = False) -> VerifyResult:
    """One verification step on top of a cache.  Does not commit."""
    draft = np.asarray(draft, dtype=np.int64)
    k = len(draft)
    parent = chain_parents(k) if parent is None else np.asarray(parent)
    depth, allowed_new = tree_depth_and_mask(parent)
    x = seq.model.embed_rows(None, np.concatenate([[pending], draft]))
    out = seq.forward_rows(x, depth, allowed_new)
    z = seq.model.logits(out)
    return _finish(z, draft, parent, log_tau, keep_logits)


def _finish(z, draft, parent, log_tau, keep_logits) -> VerifyResult:
    k = len(draft)
    tokens = np.concatenate([[-1], draft])
    path, emitted = greedy_traverse(z, tokens, parent, log_tau)
    is_chain = np.array_equal(parent, chain_parents(k))
    am, zmax, zd, gap = _row_stats(z, draft if is_chain else None)
    return VerifyResult(len(path), emitted, path, am, zmax, zd, gap, z if keep_logits else None)


def commit_step(seq: CachedSequence, res: VerifyResult) -> int:
    """KV maintenance after a step: the pending row and the accepted rows stay, everything else is rolled
    back.  Returns the new pending token (the correction or bonus token)."""
    seq.commit([0] + list(res.path))
    return res.emitted[-1]


def greedy_continuation(seq: CachedSequence, pending: int, n: int) -> List[int]:
    """n further greedy tokens after `pending` by plain one-token-per-forward decoding (the autoregressive
    baseline the method replaces).  Leaves the cache unchanged."""
    saved = ([a.copy() for a in seq.k], [a.copy() for a in seq.v])
    out, tok = [], int(pending)
    for _ in range(n):
        res = verify_cached(seq, tok, np.zeros(0, np.int64))
        tok = commit_step(seq, res)
        out.append(tok)
    seq.k, seq.v = saved
    return out


# ----------------------------------------------------------------------------- batched driver
def verify_regions(model: Decoder, caches: List[CachedSequence], pending: Sequence[int],
                   drafts: Sequence[np.ndarray], log_tau: float = 0.0) -> List[VerifyResult]:
    """Stage 1 (Eq. 2): every region's draft is verified independently; a batch is a loop."""
    return [verify_cached(c, p, d, None, log_tau) for c, p, d in zip(caches, pending, drafts)]
