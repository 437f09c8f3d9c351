"""The two-stage decode loop on the device (paper Sec. 3.1, Eq. 1-4): lane batches with retirement and hand-over,
aggregation of the Stage-1 outputs into the page draft, Stage 2.

Two independent checks.  (1) Against the library itself: with tau = 1 speculation is lossless, so on a context with a
fixed summation order the loop's outputs must equal, token for token, what plain one-token decoding through the same
library gives — whatever the drafts, the lane count or the graph batching; this exercises matching, packing, tree
verification, compaction, commit, bookkeeping and lane hand-over end to end with no tolerance.  (2) Against the oracle
loop: same inputs, same drafts; the two outputs may part only at a token the oracle chose by a near tie (top-1 / top-2
gap <= 0.1), and where they never part the per-sequence step counts and accepted totals are equal too."""
import numpy as np
import pytest

from oracle import hsd_oracle as O
from oracle import two_stage_oracle as T
from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def _library_greedy(model, prefixes, lengths, seed):
    """Plain one-token decoding through the library: the text every lossless loop must reproduce."""
    import torch
    from paper_2602_12957_b200 import runtime as R
    S = len(prefixes)
    kv = R.KvCache(model, [len(ids) + max(lengths) + 2 for _, ids in prefixes], seed=seed)    # all step together
    eng = R.Engine(model, kv, max(sum(len(ids) for _, ids in prefixes), S), S)
    first = eng.prefill([e for e, _ in prefixes], [i for _, i in prefixes])
    cu1 = eng._i32(np.arange(S + 1))
    out1 = eng.alloc_outputs(S, 1, S)
    pending, hist = first.clone(), [first.clone()]
    for _ in range(max(lengths) - 1):
        eng.verify_regions(pending, cu1, 1, S, out=out1)
        eng.commit(out1["accept_len"])
        pending = out1["emit_tokens"][:, 0].clone()
        hist.append(pending)
    eng.check_device("greedy")
    text = torch.stack(hist, 1).cpu().numpy()
    return [text[i, :lengths[i]].copy() for i in range(S)]


def _damaged(text, rng, n_err, vocab):
    d = np.asarray(text, np.int64).copy()
    for pos in rng.choice(np.arange(3, len(d)), size=min(n_err, len(d) - 3), replace=False):
        d[pos] = (d[pos] + 1 + int(rng.integers(0, vocab - 1))) % vocab
    return d.astype(np.int32)


def _setup(seed=41, n_regions=5):
    cfg = I.small_decoder(2, 8192)
    wl = I.region_workload(seed=seed, n_regions=n_regions + 1, prefix_lo=70, prefix_hi=200, draft_mean=30, draft_lo=8,
                           draft_hi=60, cfg=cfg)
    weights = I.make_weights(cfg, seed)
    prefixes = [(s.prefix_embeds, s.prefix_ids) for s in wl.seqs]
    rng = np.random.default_rng(seed)
    lengths = [int(x) for x in rng.integers(24, 70, size=n_regions)] + [90]       # regions, then the page
    return cfg, weights, prefixes, lengths, rng


@pytest.mark.parametrize("n_lanes,steps_per_poll,use_graph", [(2, 3, True), (5, 1, False), (8, 4, True)])
def test_device_loop_is_lossless_and_hands_lanes_over(n_lanes, steps_per_poll, use_graph):
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import driver as DR
    from paper_2602_12957_b200 import runtime as R
    cfg, weights, prefixes, lengths, rng = _setup()
    model = R.DeviceModel(cfg, weights, B.HSD_FLAG_DETERMINISTIC)
    text = _library_greedy(model, prefixes, lengths, seed=1)
    regions, page = prefixes[:-1], prefixes[-1]
    # the pipeline's drafts: two damaged copies of every region's text (one region gets garbage, one gets none)
    drafts = [[_damaged(t, rng, 3, cfg.vocab), _damaged(t, rng, 5, cfg.vocab)] for t in text[:-1]]
    drafts[1] = [rng.integers(0, cfg.vocab, 50).astype(np.int32)]
    drafts[2] = []
    run = DR.run_page(model, regions, drafts, lengths[:-1], page, lengths[-1], n_lanes=n_lanes, max_rows=32,
                      steps_per_poll=steps_per_poll, use_graph=use_graph, seed=3, poison=True)
    for r in range(len(regions)):
        assert run.stage1.tokens[r].tolist() == text[r].tolist(), f"region {r}"
        assert run.page_draft[r].tolist() == text[r].tolist()                       # Eq. 3: the outputs, as they are
    assert run.stage2.tokens[0].tolist() == text[-1].tolist()
    s1 = run.stage1
    assert s1.steps[1] == lengths[1] - 1 and s1.steps[2] == lengths[2] - 1          # garbage / no drafts: plain decoding
    assert s1.accepted[1] == 0 and s1.accepted[2] == 0
    for r in (0, 3, 4):                                                             # good drafts: several tokens per step
        assert s1.steps[r] < (lengths[r] - 1) * 0.6
        assert s1.accepted[r] + s1.steps[r] >= lengths[r] - 1                       # every step emits accepted + 1
    # lanes fewer than regions: the batch needs more steps than its slowest region, but far fewer than the sum
    assert s1.batch_steps >= int(s1.steps.max())
    if n_lanes < len(regions):
        assert s1.batch_steps < int(s1.steps.sum())
    print("two-stage", n_lanes, "stage1 steps", s1.steps.tolist(), "AAL", round(s1.aal, 2), "batch steps", s1.batch_steps,
          "stage2 steps", run.stage2.steps.tolist(), "ms", round(s1.ms, 2), round(run.stage2.ms, 2))


@pytest.mark.parametrize("log_tau", [0.0, float(np.log(0.75))], ids=["greedy", "tau0.75"])
def test_device_loop_follows_the_oracle_loop(log_tau):
    from paper_2602_12957_b200 import driver as DR
    from paper_2602_12957_b200 import runtime as R
    cfg, weights, prefixes, lengths, rng = _setup(seed=43, n_regions=4)
    model_o = O.Decoder(cfg, weights, np.float64)
    # drafts from the ORACLE's greedy text, so that the oracle loop accepts long runs
    regions_o = []
    for (emb, ids), n in zip(prefixes[:-1], lengths[:-1]):
        seq = O.CachedSequence(model_o)
        first = seq.prefill(emb, ids)
        text = [first] + O.greedy_continuation(seq, first, n - 1)
        regions_o.append(T.RegionInput(emb, ids, [_damaged(text, rng, 3, cfg.vocab).tolist(),
                                                  _damaged(text, rng, 4, cfg.vocab).tolist()], n))
    page_o = T.RegionInput(prefixes[-1][0], prefixes[-1][1], [], lengths[-1])
    want = T.hierarchical_decode(model_o, regions_o, page_o, n=3, max_rows=32, log_tau=log_tau)
    model = R.DeviceModel(cfg, weights, 0)
    run = DR.run_page(model, prefixes[:-1], [[np.asarray(d, np.int32) for d in r.drafts] for r in regions_o],
                      lengths[:-1], prefixes[-1], lengths[-1], n_lanes=3, max_rows=32, log_tau=log_tau, seed=5,
                      poison=True)
    checked = 0
    for r, tr in enumerate(want.region_traces):
        gaps = np.asarray(tr.token_gap)
        got = run.stage1.tokens[r].tolist()
        assert len(got) == lengths[r]
        if log_tau == 0.0:
            # the two texts may part only at a token the oracle chose by a near tie (gap <= 0.1); after that token they are
            # different texts and nothing more can be compared
            same = [a == b for a, b in zip(got, tr.tokens)]
            first_diff = same.index(False) if False in same else len(same)
            if first_diff < len(same):
                assert gaps[first_diff] <= H.GAP_EXACT, (f"region {r}: token {first_diff} differs although the oracle's "
                                                         f"choice was clear (gap {gaps[first_diff]:.3f})")
            checked += first_diff
            if first_diff == len(same):
                assert run.stage1.steps[r] == tr.steps and run.stage1.accepted[r] == sum(tr.accepted_per_step)
    if log_tau == 0.0:
        assert checked > 60, "the case must pin a fair number of tokens"
    else:
        # with a threshold the accepted text may leave the greedy path; the loop must still fill every output and
        # never take more steps than plain decoding
        assert all(run.stage1.steps[r] <= lengths[r] - 1 for r in range(len(lengths) - 1))
    assert len(run.stage2.tokens[0]) == lengths[-1]
    print("oracle loop", log_tau, want.summary(), "device stage1 steps", run.stage1.steps.tolist(), "AAL",
          round(run.stage1.aal, 2), "checked tokens", checked)


def _chain_page(cfg, order, seed, n_regions, p0=777):
    """Crops and a page for the chain decoder: the last prompt token of every crop is set so that the page's text is
    the concatenation of the regions' texts (what the method relies on)."""
    wl = I.region_workload(seed=seed, n_regions=n_regions + 1, prefix_lo=70, prefix_hi=200, draft_mean=30, draft_lo=8,
                           draft_hi=60, cfg=cfg)
    rng = np.random.default_rng(seed)
    lengths = [int(x) for x in rng.integers(20, 150, size=n_regions)]
    offs = np.concatenate([[0], np.cumsum(lengths)]).astype(int)

    def prefix(seq, pos):
        ids = seq.prefix_ids.copy()
        ids[-1] = order[pos % cfg.vocab]
        return seq.prefix_embeds, ids
    regions = [prefix(wl.seqs[i], p0 + offs[i]) for i in range(n_regions)]
    page = prefix(wl.seqs[-1], p0)
    walk = lambda start, n: order[(start + 1 + np.arange(n)) % cfg.vocab].astype(np.int32)
    texts = [walk(p0 + offs[i], lengths[i]) for i in range(n_regions)]
    return regions, page, lengths, texts, walk(p0, int(offs[-1])), rng


@pytest.mark.parametrize("log_tau", [0.0, float(np.log(0.75))], ids=["greedy", "tau0.75"])
def test_whole_hierarchy_on_a_decisive_decoder_equals_the_oracle_loop(log_tau):
    """A decoder whose every decision has a wide margin (inputs.make_chain_weights): nothing is a near tie, so the device
    loop and the oracle loop must agree on EVERYTHING — every region's text, the aggregated page draft, the page's
    text decoded in Stage 2 against that draft (no stand-in), and per sequence the number of verification steps and
    of accepted draft tokens.  The texts are also known in closed form (a walk along the decoder's token order)."""
    from paper_2602_12957_b200 import driver as DR
    from paper_2602_12957_b200 import runtime as R
    cfg = I.small_decoder(2, 8192)
    weights, order = I.make_chain_weights(cfg, 47)
    regions, page, lengths, texts, page_text, rng = _chain_page(cfg, order, 47, 5)
    drafts = [[_damaged(t, rng, max(1, len(t) // 7), cfg.vocab), _damaged(t, rng, max(1, len(t) // 5), cfg.vocab)]
              for t in texts]
    drafts[3] = [rng.integers(0, cfg.vocab, 40).astype(np.int32)]         # one region with a useless draft
    model_o = O.Decoder(cfg, weights, np.float64)
    want = T.hierarchical_decode(
        model_o, [T.RegionInput(e, i, [d.tolist() for d in ds], n) for (e, i), ds, n in zip(regions, drafts, lengths)],
        T.RegionInput(page[0], page[1], [], len(page_text)), n=3, max_rows=128, log_tau=log_tau)
    # the oracle itself against the closed form
    for tr, t in zip(want.region_traces, texts):
        assert tr.tokens == t.tolist() and min(tr.token_gap) > 10.0
    assert want.page_trace.tokens == page_text.tolist() and min(want.page_trace.token_gap) > 10.0
    model = R.DeviceModel(cfg, weights, 0)
    run = DR.run_page(model, regions, drafts, lengths, page, len(page_text), n_lanes=3, max_rows=128, log_tau=log_tau,
                      steps_per_poll=4, seed=9, poison=True)
    for r, tr in enumerate(want.region_traces):
        assert run.stage1.tokens[r].tolist() == tr.tokens, f"region {r}"
        assert run.page_draft[r].tolist() == tr.tokens
        assert int(run.stage1.steps[r]) == tr.steps, f"region {r}: steps"
        assert int(run.stage1.accepted[r]) == sum(tr.accepted_per_step), f"region {r}: accepted"
    assert run.stage2.tokens[0].tolist() == want.page_trace.tokens
    assert int(run.stage2.steps[0]) == want.page_trace.steps
    assert int(run.stage2.accepted[0]) == sum(want.page_trace.accepted_per_step)
    # Stage 2 really runs on the Stage-1 outputs: three plain steps after every region boundary, long runs between
    assert want.page_trace.steps < len(page_text) / 4
    print("decisive", log_tau, want.summary(), "device AAL", round(run.stage1.aal, 2), round(run.stage2.aal, 2))
