"""Draft-target matching and prefix-tree packing on the device (Sec. 3.2, Eq. 5-7) against the oracle: integer work,
so every output must be identical; then a device-driven decode loop (build -> tree verify -> compacting commit, no
host decision in between) against the oracle-driven one."""
import numpy as np
import pytest

from oracle import dsv_oracle as D
from oracle import hsd_oracle as O
from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def _engine():
    from paper_2602_12957_b200 import runtime as R
    wl = I.tiny_workload(n_regions=2, draft_len=8)
    weights = I.make_weights(wl.cfg, wl.seed)
    model = R.DeviceModel(wl.cfg, weights, 0)
    kv = R.KvCache(model, [400, 400], seed=1)
    return R.Engine(model, kv, 600, 2), wl, weights


def _flatten(drafts_per_seq):
    toks, off, soff = [], [0], [0]
    for drafts in drafts_per_seq:
        for d in drafts:
            toks.extend(int(t) for t in d)
            off.append(len(toks))
        soff.append(len(off) - 1)
    return (np.asarray(toks if toks else [0], np.int32), np.asarray(off, np.int32), np.asarray(soff, np.int32))


def check_build(eng, windows, drafts_per_seq, max_rows, emitted=None):
    import torch
    S, n = len(windows), len(windows[0])
    toks, off, soff = _flatten(drafts_per_seq)
    d_win = eng._i32(np.asarray(windows, np.int32).reshape(S, n)).reshape(S, n)
    em = ne = None
    acc_hist = [list(w) for w in windows]
    if emitted is not None:
        stride = max(1, max(len(e) for e in emitted))
        e = np.full((S, stride), -9, np.int32)
        for i, x in enumerate(emitted):
            e[i, :len(x)] = x
            acc_hist[i] = acc_hist[i] + list(x)
        em = eng._i32(e).reshape(S, stride)
        ne = eng._i32([len(x) for x in emitted])
    out = eng.dsv_build(d_win, eng._i32(toks), eng._i32(off), eng._i32(soff), max_rows, em, ne)
    torch.cuda.synchronize()
    q = out["q_tokens"].cpu().numpy().reshape(S, max_rows)
    p = out["parent"].cpu().numpy().reshape(S, max_rows)
    nr = out["n_rows"].cpu().numpy()
    assert out["cu_q"].cpu().numpy().tolist() == [i * max_rows for i in range(S + 1)]
    new_w = d_win.cpu().numpy()
    for i in range(S):
        hist = acc_hist[i][-n:]
        assert new_w[i].tolist() == hist
        wq, wp = ([hist[-1]], [-1]) if min(hist) < 0 else D.pack(hist, drafts_per_seq[i], n, max_rows,
                                                                 max_candidates=64)
        m = len(wq)
        assert nr[i] == m, (i, nr[i], m)
        assert q[i, :m].tolist() == wq and p[i, :m].tolist() == wp
        assert np.all(q[i, m:] == hist[-1]) and np.all(p[i, m:] == -2)
    return out


def test_build_equals_the_oracle_on_random_small_vocabularies():
    eng, _, _ = _engine()
    rng = np.random.default_rng(17)
    for case in range(40):
        S = int(rng.integers(1, 5))
        n = int(rng.integers(1, 5))
        vocab = int(rng.integers(2, 6))
        max_rows = int(rng.choice([128, 128, 40, 9, 2, 1]))
        windows = [rng.integers(0, vocab, size=n).tolist() for _ in range(S)]
        drafts = [[rng.integers(0, vocab, size=int(rng.integers(0, 300))).tolist()
                   for _ in range(int(rng.integers(0, 4)))] for _ in range(S)]
        emitted = None
        if case % 3 == 1:
            emitted = [rng.integers(0, vocab, size=int(rng.integers(0, 7))).tolist() for _ in range(S)]
        check_build(eng, windows, drafts, max_rows, emitted)


def test_build_edge_cases():
    eng, _, _ = _engine()
    # the window is not full yet: no matching, bare root
    check_build(eng, [[-1, 4, 5]], [[[4, 5, 6, 7]]], 128)
    # the paper's shape of example: three candidates sharing their first token
    check_build(eng, [[1, 2, 3]], [[[0, 1, 2, 3, 10, 11, 12], [1, 2, 3, 10, 13], [9, 9, 1, 2, 3, 10, 14, 1, 2, 3]]], 128)
    # a match at the very end of a draft has an empty suffix and gives no candidate
    check_build(eng, [[1, 2, 3]], [[[7, 1, 2, 3]]], 128)
    # more matches than candidates are kept, a long draft (several passes of the CTA), one repeated token
    check_build(eng, [[5, 5]], [[[5] * 5000]], 128)
    check_build(eng, [[5, 5]], [[(list(range(6, 40)) + [5, 5]) * 90 + [8]]], 128)
    # sequences without drafts beside sequences with drafts
    check_build(eng, [[1, 2], [1, 2], [3, 4]], [[], [[1, 2, 3, 4, 5]], [[3, 4]]], 16)


def test_malformed_draft_offsets_are_clamped_not_followed():
    """Offsets that point outside the draft arrays shorten or drop drafts (as if the arrays ended there); the call
    stays inside the arrays and its outputs are well-formed trees."""
    import torch
    eng, _, _ = _engine()
    toks = eng._i32([1, 2, 3, 4, 5, 1, 2, 3, 9, 9])
    window = eng._i32(np.asarray([[1, 2, 3]], np.int32)).reshape(1, 3)
    for off, soff in (([0, 5, 1 << 30], [0, 2]), ([-7, 5, 10], [0, 2]), ([0, 5, 10], [0, 1 << 20]),
                      ([8, 3, 10], [0, 2]), ([0, 5, 10], [-3, 2])):
        out = eng.dsv_build(window, toks, eng._i32(off), eng._i32(soff), 16)
        torch.cuda.synchronize()
        n = int(out["n_rows"][0])
        par = out["parent"].cpu().numpy()[:16]
        assert 1 <= n <= 16 and par[0] == -1 and all(0 <= par[r] < r for r in range(1, n)) and all(par[n:] == -2)


def test_device_driven_loop_follows_the_oracle_driven_loop():
    """Three decode steps per sequence with no host decision in between on the device side: hsd_dsv_build (fed by the
    previous step's emitted tokens) -> hsd_verify_tree -> hsd_kv_commit_tree.  The oracle side makes the same steps
    with its own matching, verification and commits.  Compared: every packed tree (exact while the emitted histories
    agree), every row's logits, and the emitted tokens wherever the oracle's decisions are clear."""
    import torch
    from paper_2602_12957_b200 import runtime as R
    wl = I.tiny_workload(n_regions=3, draft_len=8)
    cfg = wl.cfg
    weights = I.make_weights(cfg, wl.seed)
    model_o = O.Decoder(cfg, weights, np.float64)
    S, n, ROWS, STEPS = len(wl.seqs), 3, 32, 3
    caches, hist, drafts = [], [], []
    rng = np.random.default_rng(4)
    for i, s in enumerate(wl.seqs):
        c = O.CachedSequence(model_o)
        p = c.prefill(s.prefix_embeds, s.prefix_ids)
        # the "pipeline drafts": the oracle's own greedy text with substitution errors, twice, differently damaged
        g = [p] + O.greedy_continuation(c, p, 40)
        d1, d2 = list(g), list(g)
        for pos in (9 + i, 20, 31):
            d1[pos] = (d1[pos] + 1) % cfg.vocab
        for pos in (14, 26 + i):
            d2[pos] = (d2[pos] + 7) % cfg.vocab
        drafts.append([d1, d2])
        caches.append(c)
        hist.append(list(g[:1]))
    # plain decode steps until n tokens are accepted, so that a full window exists
    for i in range(S):
        c = caches[i]
        while len(hist[i]) < n:
            r = O.verify_cached(c, hist[i][-1], [])
            c.commit([0])
            hist[i].append(int(r.emitted[0]))
    # device: prefill, the same plain steps
    model = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(model, [s.prefix_len + 200 for s in wl.seqs], seed=2, poison=True)
    eng = R.Engine(model, kv, max(sum(s.prefix_len for s in wl.seqs), 2 * S * ROWS), S)
    first = eng.prefill([s.prefix_embeds for s in wl.seqs], [s.prefix_ids for s in wl.seqs])
    cu1 = eng._i32(np.arange(S + 1))
    pend = first.clone()
    dev_hist = [[int(x)] for x in first.cpu().tolist()]
    for _ in range(n - 1):
        o1 = eng.verify_regions(pend, cu1, 1, S)
        eng.commit(o1["accept_len"])
        pend = o1["emit_tokens"][:, 0].clone()
        for i, x in enumerate(pend.cpu().tolist()):
            dev_hist[i].append(int(x))
    eng.check_device("plain steps")
    if dev_hist != hist:
        pytest.skip("a near tie split the two sides before the loop started")
    toks, off, soff = _flatten(drafts)
    d_toks, d_off, d_soff = eng._i32(toks), eng._i32(off), eng._i32(soff)
    window = eng._i32(np.asarray([h[-n:] for h in hist], np.int32).reshape(S, n)).reshape(S, n)
    emit = n_emit = None
    bout = vout = None
    live = [True] * S
    compared = 0
    for step in range(STEPS):
        bout = eng.dsv_build(window, d_toks, d_off, d_soff, ROWS, emit, n_emit, out=bout)
        vout = eng.verify_tree(bout["q_tokens"], bout["cu_q"], bout["parent"], ROWS, S * ROWS, out=vout)
        eng.commit_tree(vout["accept_len"], vout["accept_rows"])
        eng.check_device(f"loop step {step}")
        emit, n_emit = vout["emit_tokens"], vout["n_emit"]
        torch.cuda.synchronize()
        q = bout["q_tokens"].cpu().numpy().reshape(S, ROWS)
        par = bout["parent"].cpu().numpy().reshape(S, ROWS)
        nr = bout["n_rows"].cpu().numpy()
        g_emit = vout["emit_tokens"].cpu().numpy()
        g_ne = vout["n_emit"].cpu().numpy()
        zm = vout["row_zmax"].cpu().numpy().reshape(S, ROWS)
        for i in range(S):
            if not live[i]:
                continue
            wq, wp = D.pack(hist[i], drafts[i], n, ROWS)
            m = len(wq)
            assert nr[i] == m and q[i, :m].tolist() == wq and par[i, :m].tolist() == wp, f"step {step} seq {i}: tree"
            res = O.verify_cached(caches[i], wq[0], np.asarray(wq[1:], np.int64), np.asarray(wp, np.int64), 0.0,
                                  keep_logits=True)
            assert np.all(np.abs(zm[i, :m] - res.row_zmax) <= H.LOGIT_TOL), f"step {step} seq {i}: zmax"
            compared += m
            caches[i].commit([0] + list(res.path))
            hist[i] += [int(t) for t in res.emitted]
            got = g_emit[i, :g_ne[i]].tolist()
            clear = all(res.row_gap[r] > H.GAP_EXACT for r in [0] + list(res.path))
            if got != [int(t) for t in res.emitted]:
                assert not clear, f"step {step} seq {i}: emitted {got} vs {res.emitted} on clear rows"
                live[i] = False                    # a tolerated near tie: the two histories part here
    assert compared > 0
