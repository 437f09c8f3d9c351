"""Parity at the benchmark's full size and launch configuration: the 24-layer decoder, all 16 regions of the
region-level workload in one verify call, with the CPU oracle (float32) run on a sample of the regions it can finish
in about a minute.  The sampled regions' drafts are planted along the oracle's greedy path; the others carry random
drafts (their results are checked for internal consistency only)."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def test_region_stage_full_size_sampled_rows_match_oracle():
    cfg = I.DECODER
    wl = I.region_workload(seed=I.BASE_SEED + 1, cfg=cfg)
    weights = I.make_weights(cfg, I.BASE_SEED + 1)
    sample = sorted(range(len(wl.seqs)), key=lambda i: wl.seqs[i].prefix_len + wl.seqs[i].draft_len)[:2]
    orc = H.oracle_regions(wl, weights, np.float32, which=sample)
    rng = np.random.default_rng(0)
    pend = {i: (orc[i].pending if i in orc else int(rng.integers(0, cfg.vocab))) for i in range(len(wl.seqs))}
    drafts = {i: (orc[i].draft if i in orc else wl.seqs[i].rand_tokens[:wl.seqs[i].draft_len]) for i in range(len(wl.seqs))}
    per, eng, (toks, cu, total_q) = H.gpu_regions(wl, weights, pend, drafts, 0)
    assert total_q == sum(s.draft_len + 1 for s in wl.seqs)
    stats = {}
    for i in sample:
        o, g = orc[i], per[i]
        H.check_first_token(f"seq{i}", o, g["first_token"])
        H.compare_rows(f"seq{i}", o.res, o.draft, g["row_argmax"], g["row_zmax"], g["row_zdraft"], stats)
        H.compare_sequence(f"seq{i}", o.res, o.draft, g["accept_len"], g["emit"], g["n_emit"], g["row_argmax"], stats)
    for i in range(len(wl.seqs)):            # every sequence: the decision is consistent with the row argmaxes
        g, d = per[i], drafts[i]
        a = int(g["accept_len"])
        assert 0 <= a <= len(d) and int(g["n_emit"]) == a + 1
        assert all(g["row_argmax"][j] == d[j] for j in range(a)) and (a == len(d) or g["row_argmax"][a] != d[a])
        assert g["emit"][a] == g["row_argmax"][a] and np.all(np.isfinite(g["row_zmax"]))
    print("full size", sample, stats, [(len(orc[i].draft), orc[i].res.accept_len) for i in sample])
    assert stats["max_dz"] < H.LOGIT_TOL


def test_tree_step_full_size_sampled_rows_match_oracle():
    """The tree workload's shape (24 layers, 16 regions x 128 packed rows in one hsd_verify_tree call, tau = 0.75):
    the region with the shortest prefix is checked row by row against the float32 oracle, every other region for
    consistency between its path and its own rows."""
    import torch
    from oracle import hsd_oracle as O
    from paper_2602_12957_b200 import runtime as R
    from .test_gpu_tree import LOG_TAU_PAPER, oracle_decisive_steps, traverse_rows
    cfg = I.DECODER
    wl = I.region_workload(seed=I.BASE_SEED + 1, cfg=cfg)
    weights = I.make_weights(cfg, I.BASE_SEED + 1)
    S, NODES = len(wl.seqs), 127
    pick = min(range(S), key=lambda i: wl.seqs[i].prefix_len)
    model_o = O.Decoder(cfg, weights, np.float32)
    cache = O.CachedSequence(model_o)
    sp = wl.seqs[pick]
    pending_o = cache.prefill(sp.prefix_embeds if np.any(sp.prefix_ids < 0) else None, sp.prefix_ids)
    greedy = O.greedy_continuation(cache, pending_o, 25)
    rng = np.random.default_rng(3)
    toks_l, par_l, pend = [], [], []
    for i in range(S):
        if i == pick:
            t, p, _ = I.plant_tree(greedy, NODES, 24, cfg.vocab, 1000 + i, n_branches=8)
            pend.append(pending_o)
        else:
            t, p, _ = I.plant_tree(rng.integers(0, cfg.vocab, size=NODES).tolist(), NODES, 0, cfg.vocab, 1000 + i)
            pend.append(int(rng.integers(0, cfg.vocab)))
        toks_l.append(t); par_l.append(p)
    res = O.verify_cached(cache, pending_o, toks_l[pick], par_l[pick], LOG_TAU_PAPER, keep_logits=True)
    model = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(model, [s.prefix_len + 2 * (NODES + 1) + 16 for s in wl.seqs], seed=5, poison=True)
    T = S * (NODES + 1)
    eng = R.Engine(model, kv, max(sum(s.prefix_len for s in wl.seqs), 2 * T), S)
    first = eng.prefill([s.prefix_embeds if np.any(s.prefix_ids < 0) else None for s in wl.seqs],
                        [s.prefix_ids for s in wl.seqs])
    eng.check_device("prefill")
    toks, cu = I.pack_queries(pend, toks_l)
    parent = np.concatenate(par_l).astype(np.int32)
    out = eng.verify_tree(eng._i32(toks), eng._i32(cu), eng._i32(parent), NODES + 1, T, log_tau=LOG_TAU_PAPER)
    eng.check_device("verify_tree")
    torch.cuda.synchronize()
    host = {n: t.cpu().numpy() for n, t in out.items()}
    for i in range(S):
        a, b = int(cu[i]), int(cu[i + 1])
        tokens = np.concatenate([[-1], toks_l[i]])
        am, zm, zc = host["row_argmax"][a:b], host["row_zmax"][a:b], host["row_zchild"][a:b]
        assert np.all(np.isfinite(zm)) and np.all(np.isfinite(zc[1:]))
        g_acc = int(host["accept_len"][i])
        want_path, want_emit = traverse_rows(par_l[i], tokens, am, zm, zc, LOG_TAU_PAPER)
        assert host["accept_rows"][i][:g_acc].tolist() == want_path
        assert host["emit_tokens"][i][:g_acc + 1].tolist() == want_emit
        if i == pick:
            dz = np.abs(zm - res.row_zmax)
            dc = max(abs(zc[j] - res.logits[par_l[i][j], int(tokens[j])]) for j in range(1, b - a))
            assert dz.max() <= H.LOGIT_TOL and dc <= H.LOGIT_TOL, (dz.max(), dc)
            for j in range(b - a):
                if res.row_gap[j] > H.GAP_EXACT:
                    assert am[j] == res.row_argmax[j]
            clear = oracle_decisive_steps(res, par_l[i], tokens, LOG_TAU_PAPER)
            m = min(clear, len(res.path))
            assert want_path[:m] == list(res.path)[:m]
            print("full-size tree", pick, "max dz", float(dz.max()), "max dzchild", float(dc), "oracle path", len(res.path),
                  "clear decisions", clear, "library path", g_acc)


# ------------------------------------------------------------------------------------------------------------------
# The page-level, long-document and mixed configurations at their full sizes (24 layers, the benchmark's launch
# configuration: default GEMM tiles, default attention plan).  Rows are teacher-forced, so random drafts serve: every
# row's argmax, maximum and draft-token logit is well defined whatever the draft is, and the oracle needs one float32
# prefill and one verify pass per sampled sequence (no greedy continuation on the CPU).
def _oracle_sequence(cfg, weights, seq):
    from oracle import hsd_oracle as O
    model = O.Decoder(cfg, weights, np.float32)
    cache = O.CachedSequence(model)
    emb = seq.prefix_embeds if np.any(seq.prefix_ids < 0) else None
    first = cache.prefill(emb, seq.prefix_ids)
    return cache, first


def _check_chunk(tag, res, draft, g, stats):
    k = len(draft)
    H.compare_rows(tag, res, draft, g["row_argmax"][:k + 1], g["row_zmax"][:k + 1], g["row_zdraft"][:k + 1], stats)
    H.compare_sequence(tag, res, draft, g["accept_len"], g["emit"], g["n_emit"], g["row_argmax"][:k + 1], stats)


def _page_outputs(out):
    g = {k: v.cpu().numpy() for k, v in out.items()}
    return {"row_argmax": g["row_argmax"], "row_zmax": g["row_zmax"], "row_zdraft": g["row_zdraft"],
            "accept_len": g["accept_len"][0], "n_emit": g["n_emit"][0], "emit": g["emit_tokens"][0]}


def test_page_stage_full_size_two_chunks_with_commit_match_oracle():
    """Page-level stage: prefix of 4,096 visual rows + 256 prompt tokens, a 512-token chunk through hsd_verify_page,
    a commit of 300 accepted tokens (the rest rolled back), then a second 512-token chunk on top of it."""
    import torch
    from oracle import hsd_oracle as O
    from paper_2602_12957_b200 import runtime as R
    cfg = I.DECODER
    wl = I.page_workload(cfg=cfg)
    s = wl.seqs[0]
    weights = I.make_weights(cfg, I.BASE_SEED + 1)
    cache, first_o = _oracle_sequence(cfg, weights, s)
    dm = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(dm, [s.prefix_len + 2 * 513 + 64], seed=wl.seed, poison=True)
    eng = R.Engine(dm, kv, s.prefix_len, 1)
    first = eng.prefill([s.prefix_embeds], [s.prefix_ids])
    eng.check_device("prefill")
    pl = np.sort(cache.last_prefill_logits)
    if pl[-1] - pl[-2] > H.GAP_EXACT:
        assert int(first[0].item()) == first_o
    stats = {}
    pending, keep = first_o, 300
    for n, chunk in enumerate((s.rand_tokens[:512], s.rand_tokens[512:1024])):
        res = O.verify_cached(cache, pending, chunk, keep_logits=True)
        out = eng.verify_page(0, torch.tensor([pending], dtype=torch.int32, device=eng.dev), eng._i32(chunk))
        eng.check_device("verify_page")
        _check_chunk(f"page chunk {n}", res, chunk, _page_outputs(out), stats)
        # both sides keep the pending row and 300 draft rows (a caller-chosen length), everything after is rolled back
        eng.commit(torch.tensor([keep], dtype=torch.int32, device=eng.dev))
        cache.commit(range(keep + 1))
        assert int(kv.seq_lens[0].item()) == cache.length == s.prefix_len + (n + 1) * (keep + 1)
        pending = int(chunk[keep])
    print("full-size page", stats)
    assert stats["max_dz"] < H.LOGIT_TOL and stats["exact_rows"] > 200


def test_mixed_batch_full_size_sampled_sequences_match_oracle():
    """Mixed serving batch: 64 regions and two 1,024-token page chunks over 4,352-token prefixes in ONE
    hsd_verify_regions call (66 sequences); the oracle runs on the two cheapest regions and on one page chunk."""
    from oracle import hsd_oracle as O
    cfg = I.DECODER
    wl = I.mixed_workload(cfg=cfg)
    weights = I.make_weights(cfg, I.BASE_SEED + 1)
    S = len(wl.seqs)
    assert S == 66
    regions = sorted(range(64), key=lambda i: wl.seqs[i].prefix_len + 8 * wl.seqs[i].draft_len)[:2]
    sample = regions + [64]
    rng = np.random.default_rng(1)
    pend = {i: int(rng.integers(0, cfg.vocab)) for i in range(S)}
    drafts = {i: wl.seqs[i].rand_tokens[:wl.seqs[i].draft_len] for i in range(S)}
    orc = {}
    for i in sample:
        cache, first_o = _oracle_sequence(cfg, weights, wl.seqs[i])
        pend[i] = first_o
        orc[i] = (O.verify_cached(cache, first_o, drafts[i], keep_logits=True), cache)
    per, eng, (toks, cu, total_q) = H.gpu_regions(wl, weights, pend, drafts, 0)
    assert total_q == sum(s.draft_len + 1 for s in wl.seqs) and int(np.diff(cu).max()) == 1025
    stats = {}
    for i in sample:
        res, cache = orc[i]
        pl = np.sort(cache.last_prefill_logits)
        if pl[-1] - pl[-2] > H.GAP_EXACT:
            assert per[i]["first_token"] == pend[i]
        _check_chunk(f"mixed seq{i}", res, drafts[i], per[i], stats)
    for i in range(S):                       # every sequence: decision consistent with its own rows, logits finite
        g, d = per[i], drafts[i]
        a = int(g["accept_len"])
        assert 0 <= a <= len(d) and int(g["n_emit"]) == a + 1
        assert all(g["row_argmax"][j] == d[j] for j in range(a)) and (a == len(d) or g["row_argmax"][a] != d[a])
        assert g["emit"][a] == g["row_argmax"][a] and np.all(np.isfinite(g["row_zmax"]))
    print("full-size mixed", sample, stats)
    assert stats["max_dz"] < H.LOGIT_TOL
