"""Pins for the two-stage decode loop oracle (Sec. 3.1, Eq. 1-4): fixed by properties that do not depend on it —
exact-match speculation is lossless (the output is the plain greedy continuation whatever the drafts), the closed-form
step count when the draft is the model's own text, the paper's printed steps-per-token identity, and the wiring of
Stage 1 into Stage 2."""
import math
import os

import numpy as np
import pytest

from oracle import dsv_oracle as D
from oracle import hsd_oracle as O
from oracle import two_stage_oracle as T
from paper_2602_12957_b200 import inputs as I

SMALL = I.ModelConfig(n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=128, vocab=97)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_numbers.txt")


def model_and_prefix(seed, n=14, n_visual=6):
    model = O.Decoder(SMALL, I.make_weights(SMALL, seed), np.float64)
    rng = np.random.default_rng(seed)
    emb = np.zeros((n, SMALL.d_model), np.float32)
    emb[:n_visual] = rng.standard_normal((n_visual, SMALL.d_model)).astype(np.float32)
    ids = np.full(n, -1, np.int64)
    ids[n_visual:] = rng.integers(0, SMALL.vocab, n - n_visual)
    return model, emb, ids


def greedy_text(model, emb, ids, length):
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    return [first] + O.greedy_continuation(seq, first, length - 1)


def damaged(text, rng, n_err, vocab):
    d = list(text)
    for pos in rng.choice(np.arange(3, len(d)), size=n_err, replace=False):
        d[pos] = (d[pos] + 1 + int(rng.integers(0, vocab - 1))) % vocab
    return d


@pytest.mark.parametrize("drafts_kind", ["none", "own_text", "damaged", "garbage", "two_damaged"])
def test_exact_match_speculation_is_lossless(drafts_kind):
    """tau = 1: whatever the draft set, SpecDecode returns the decoder's own greedy continuation."""
    model, emb, ids = model_and_prefix(5)
    text = greedy_text(model, emb, ids, 60)
    rng = np.random.default_rng(1)
    drafts = {"none": [], "own_text": [text], "damaged": [damaged(text, rng, 5, SMALL.vocab)],
              "garbage": [list(rng.integers(0, SMALL.vocab, 80))],
              "two_damaged": [damaged(text, rng, 4, SMALL.vocab), damaged(text, rng, 6, SMALL.vocab)]}[drafts_kind]
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    tr = T.spec_decode(seq, first, drafts, 60, n=3, max_rows=16)
    assert tr.tokens == text
    assert seq.length == len(ids) + sum(a + 1 for a in tr.accepted_per_step)       # pending + accepted rows per step
    if drafts_kind in ("none", "garbage"):
        assert tr.steps == 59 and tr.aal == 0.0                                    # plain decoding: one token per step
    if drafts_kind != "none" and drafts_kind != "garbage":
        assert tr.steps < 40 and tr.aal > 0.5


def simulate_steps(text, drafts, n, max_rows):
    """Steps of a lossless (tau = 1) decode whose output is known to be `text`, without any decoder: pack the tree
    from the accepted tokens, follow the known text through it as far as it goes, append that run plus one token."""
    out, accepted, rows = [text[0]], [], []
    while len(out) < len(text):
        q, par = D.pack(out, drafts, n, max_rows)
        s, a = 0, 0
        while len(out) + a < len(text):
            want = text[len(out) + a]
            kids = [r for r in range(1, len(q)) if par[r] == s and q[r] == want]
            if not kids:
                break
            s, a = kids[0], a + 1
        room = len(text) - len(out)
        out.extend(text[len(out):len(out) + a + 1])
        accepted.append(min(a, room))
        rows.append(len(q))
    return accepted, rows


@pytest.mark.parametrize("kind", ["own_text", "damaged", "two_damaged"])
@pytest.mark.parametrize("max_rows", [8, 128])
def test_step_sequence_equals_a_decoder_free_simulation(kind, max_rows):
    """Under tau = 1 the output is the greedy text, so how far each step gets is a question about the packed tree
    alone; the loop (window, packing, commit, next pending token) must reproduce that step by step."""
    model, emb, ids = model_and_prefix(10)
    text = greedy_text(model, emb, ids, 120)
    rng = np.random.default_rng(5)
    drafts = {"own_text": [text], "damaged": [damaged(text, rng, 10, SMALL.vocab)],
              "two_damaged": [damaged(text, rng, 8, SMALL.vocab), damaged(text[20:], rng, 8, SMALL.vocab)]}[kind]
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    tr = T.spec_decode(seq, first, drafts, 120, n=3, max_rows=max_rows)
    accepted, rows = simulate_steps(text, drafts, 3, max_rows)
    assert tr.tokens == text
    assert tr.accepted_per_step == accepted and tr.rows_per_step == rows


@pytest.mark.parametrize("max_rows", [4, 8])
def test_own_text_as_draft_gives_the_closed_form_step_count(max_rows):
    """Draft = the decoder's own text, tau = 1, no window occurring twice: the first n - 1 steps have no full window
    and emit one token each; from then on every step accepts max_rows - 1 draft tokens and adds the bonus token."""
    n, length = 3, 24
    model, emb, ids = model_and_prefix(16)
    text = greedy_text(model, emb, ids, length)
    windows = [tuple(text[i:i + n]) for i in range(len(text) - n + 1)]
    assert len(set(windows)) == len(windows)              # (this seed's text has no repeated window this early)
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    tr = T.spec_decode(seq, first, [text], length, n=n, max_rows=max_rows)
    assert tr.tokens == text
    assert tr.steps == (n - 1) + math.ceil((length - n) / max_rows)
    assert tr.accepted_per_step[:n - 1] == [0] * (n - 1)
    assert all(a == max_rows - 1 for a in tr.accepted_per_step[n - 1:-1])
    assert all(r == max_rows for r in tr.rows_per_step[n - 1:-1])


def test_steps_per_token_identity_and_printed_numbers():
    """Every step emits its accepted tokens plus one: forward passes per emitted token = 1 / (AAL + 1).  The paper
    prints AAL 4.55 beside a forward-pass ratio of 0.179 (supplement), which this identity reproduces."""
    model, emb, ids = model_and_prefix(7)
    text = greedy_text(model, emb, ids, 90)
    rng = np.random.default_rng(2)
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    tr = T.spec_decode(seq, first, [damaged(text, rng, 9, SMALL.vocab)], 90, n=3, max_rows=32)
    emitted = len(tr.tokens) - 1
    assert 0 <= tr.steps * (tr.aal + 1.0) - emitted <= 1 + 1e-9           # the last step may be cut by the budget
    printed = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            printed[k.strip()] = float(v)
    assert abs(1.0 / (printed["aal_hunyuanocr"] + 1.0) - printed["forward_pass_ratio"]) < 2e-3


def test_stage_two_verifies_the_stage_one_outputs():
    """Eq. 2-4: regions decode independently from their own drafts; the page draft is exactly the set of their
    outputs; with tau = 1 the page output is the page's own greedy text, reached in fewer steps than tokens because
    the region outputs (here: pieces of the page text) are matched and accepted in runs."""
    model, emb, ids = model_and_prefix(8, n=20, n_visual=10)
    page_text = greedy_text(model, emb, ids, 80)
    rng = np.random.default_rng(3)
    regions = []
    for i, (a, b) in enumerate(((0, 30), (25, 55), (50, 80))):
        # a region crop = its own visual rows; its pipeline draft = the page's text of that span, damaged
        r_emb = rng.standard_normal((8, SMALL.d_model)).astype(np.float32)
        regions.append(T.RegionInput(r_emb, np.full(8, -1, np.int64), [damaged(page_text[a:b], rng, 2, SMALL.vocab)], 24))
    res = T.hierarchical_decode(model, regions, T.RegionInput(emb, ids, [], 80), n=3, max_rows=32)
    for r, tr in zip(regions, res.region_traces):
        seq = O.CachedSequence(model)
        first = seq.prefill(r.prefix_embeds, r.prefix_ids)
        assert tr.tokens == [first] + O.greedy_continuation(seq, first, r.max_new - 1)     # lossless per region
    assert res.page_draft == [t.tokens for t in res.region_traces]
    assert res.page_trace.tokens == page_text
    s = res.summary()
    assert s["stage2_tokens"] == 80 and s["stage2_steps"] == res.page_trace.steps <= 79
    # the same page with its own text among the drafts needs far fewer steps than plain decoding
    seq = O.CachedSequence(model)
    first = seq.prefill(emb, ids)
    good = T.spec_decode(seq, first, [page_text[10:70]], 80, n=3, max_rows=32)
    assert good.tokens == page_text and good.steps < 30


def test_thresholded_acceptance_accepts_at_least_as_much():
    """tau < 1 only ever extends a step's accepted path relative to tau = 1 on the same state."""
    model, emb, ids = model_and_prefix(9)
    text = greedy_text(model, emb, ids, 40)
    rng = np.random.default_rng(4)
    d = damaged(text, rng, 6, SMALL.vocab)
    out = text[:5]
    q, par = D.pack(out, [d], 3, 32)
    seq = O.CachedSequence(model)
    seq.prefill(emb, ids)
    # bring the cache to the state after out[:4]
    for t_ in out[:4]:
        r_ = O.verify_cached(seq, t_, np.zeros(0, np.int64))
        O.commit_step(seq, r_)
    strict = O.verify_cached(seq, q[0], np.asarray(q[1:]), np.asarray(par), 0.0)
    loose = O.verify_cached(seq, q[0], np.asarray(q[1:]), np.asarray(par), float(np.log(0.05)))
    assert loose.accept_len >= strict.accept_len
    assert loose.path[:strict.accept_len] == strict.path


def test_chain_decoder_page_text_is_the_concatenation_and_stage2_step_count_is_closed_form():
    """On the chain decoder (inputs.make_chain_weights) every text is a known walk along the token order, the page's
    text is the concatenation of the regions' texts, and all tokens of the walk are distinct, so Stage 2's course is
    fixed by the window rule alone.  The first token of region i's part of the page comes for free (the prefill's
    token for i = 0, else the bonus token of the step that accepted the end of draft i - 1); two plain steps bring
    the next two; then the window (n = 3) lies inside draft i and the remaining len_i - 3 tokens go 127 accepted + 1
    bonus per step: ceil((len_i - 3) / 128) steps, as long as len_i >= 4 and (len_i - 3) is no multiple of 128 (then
    the last bonus token would still belong to part i)."""
    cfg = I.small_decoder(1, 4096)
    weights, order = I.make_chain_weights(cfg, 11)
    model = O.Decoder(cfg, weights, np.float64)
    rng = np.random.default_rng(11)
    lengths = [30, 140, 7, 300]
    offs = np.concatenate([[0], np.cumsum(lengths)]).astype(int)
    p0 = 50

    def prefix(pos, L):
        emb = I.bf16_round(rng.standard_normal((L, cfg.d_model)).astype(np.float32))
        ids = np.full(L, -1, np.int32)
        ids[-4:] = order[[5, 6, 7, pos % cfg.vocab]]
        return emb, ids
    walk = lambda start, n: order[(start + 1 + np.arange(n)) % cfg.vocab].tolist()
    regions = []
    for i, n in enumerate(lengths):
        e, ids = prefix(p0 + offs[i], 20 + 3 * i)
        regions.append(T.RegionInput(e, ids, [walk(p0 + offs[i], n)], n))        # exact drafts
    e, ids = prefix(p0, 33)
    res = T.hierarchical_decode(model, regions, T.RegionInput(e, ids, [], int(offs[-1])), n=3, max_rows=128)
    for i, tr in enumerate(res.region_traces):
        assert tr.tokens == walk(p0 + offs[i], lengths[i])
    assert res.page_draft == [walk(p0 + offs[i], n) for i, n in enumerate(lengths)]
    assert res.page_trace.tokens == walk(p0, int(offs[-1]))
    want_steps = sum(2 + -(-(n - 3) // 128) for n in lengths)
    assert res.page_trace.steps == want_steps, (res.page_trace.steps, want_steps, res.page_trace.accepted_per_step)
