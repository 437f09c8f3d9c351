"""GPU parity of candidate-tree verification (paper Sec. 3.2: prefix tree of Eq. 7 packed into one sequence, the
tree-ancestry mask of Fig. 2(c), greedy traversal of Eq. 9-12) through the C-ABI against the CPU oracle, including
the KV maintenance afterwards (the accepted path's rows are compacted, checked by a second step on top of it)."""
import numpy as np
import pytest

from oracle import hsd_oracle as O
from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu

LOG_TAU_PAPER = float(np.log(0.75))      # tau = 0.75 (Sec. 4.3)


def traverse_rows(parent, tokens, argmax, zmax, zchild, log_tau):
    """The traversal rule of Eq. 9-12 restated over per-row summaries (what the library returns): used to check
    that the library's path is consistent with its own row outputs."""
    n = len(parent)
    s, path = 0, []
    while True:
        kids = [j for j in range(1, n) if parent[j] == s]
        if not kids:
            break
        if log_tau == 0.0:
            hit = [j for j in kids if tokens[j] == argmax[s]]
            if not hit:
                break
            nxt = hit[0]
        else:
            nxt = max(kids, key=lambda j: (zchild[j], -int(tokens[j])))
            if not (np.float32(zchild[nxt]) - np.float32(zmax[s]) >= np.float32(log_tau)):
                break
        path.append(nxt)
        s = nxt
    return path, [int(tokens[j]) for j in path] + [int(argmax[s])]


def oracle_decisive_steps(res, parent, tokens, log_tau):
    """How many decisions of the oracle's traversal, from the root on, are further than the tolerance from
    flipping.  len(path) + 1 means every move and the final stop (with its emitted token) are clear."""
    z = res.logits
    n = len(parent)
    s = 0
    clear = 0
    for nxt in list(res.path) + [None]:
        if res.row_gap[s] <= H.GAP_EXACT:              # u_hat itself (the token a child must match / the emitted one)
            return clear
        if log_tau != 0.0:
            kids = [j for j in range(1, n) if parent[j] == s]
            if kids:
                sc = sorted((z[s, int(tokens[j])] for j in kids), reverse=True)
                if len(sc) > 1 and sc[0] - sc[1] <= H.GAP_EXACT:
                    return clear
                if abs(sc[0] - z[s].max() - log_tau) <= H.GAP_EXACT:
                    return clear
        clear += 1
        if nxt is None:
            break
        s = nxt
    return clear


def run_tree_case(wl, n_nodes, log_tau, flags=0, second_step=True, shuffle=True, chain=False):
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = wl.cfg
    weights = I.make_weights(cfg, wl.seed)
    model_o = O.Decoder(cfg, weights, np.float64)
    S = len(wl.seqs)
    # ---- oracle: prefill, greedy continuation, planted tree, verification
    caches, pend, toks_l, par_l, res_l = [], [], [], [], []
    for i, s in enumerate(wl.seqs):
        cache = O.CachedSequence(model_o)
        emb = s.prefix_embeds if np.any(s.prefix_ids < 0) else None
        p = cache.prefill(emb, s.prefix_ids)
        k = n_nodes[i]
        greedy = O.greedy_continuation(cache, p, k) if k else []
        if chain:
            t = I.plant_draft(greedy, k, s.agree_len % (k + 1), s.rand_tokens, cfg.vocab, False) if k else np.zeros(0, np.int32)
            par = O.chain_parents(k).astype(np.int32)
        else:
            t, par, _ = I.plant_tree(greedy, k, s.agree_len % (k + 1), cfg.vocab, wl.seed + i, shuffle=shuffle)
        res = O.verify_cached(cache, p, t, par, log_tau, keep_logits=True)
        caches.append(cache); pend.append(p); toks_l.append(t); par_l.append(par); res_l.append(res)
    # ---- library
    model = R.DeviceModel(cfg, weights, flags)
    caps = [s.prefix_len + 2 * (n_nodes[i] + 1) + 80 for i, s in enumerate(wl.seqs)]
    kv = R.KvCache(model, caps, seed=3, poison=True)
    total_q = sum(n_nodes) + S
    max_q = max(n_nodes) + 1
    eng = R.Engine(model, kv, max(sum(s.prefix_len for s in wl.seqs), 2 * total_q), S)
    first = eng.prefill([s.prefix_embeds if np.any(s.prefix_ids < 0) else None for s in wl.seqs],
                        [s.prefix_ids for s in wl.seqs])
    eng.check_device("prefill")
    toks, cu = I.pack_queries(pend, toks_l)
    parent = np.concatenate(par_l).astype(np.int32)
    out = eng.verify_tree(eng._i32(toks), eng._i32(cu), eng._i32(parent), max_q, total_q, log_tau=log_tau)
    eng.check_device("verify_tree")
    torch.cuda.synchronize()
    host = {n: t.cpu().numpy() for n, t in out.items()}
    stats = {"exact": 0, "tolerated": 0, "max_dz": 0.0}
    for i in range(S):
        a, b = int(cu[i]), int(cu[i + 1])
        res, par, t = res_l[i], par_l[i], toks_l[i]
        n = b - a
        tokens = np.concatenate([[-1], t])
        am, zm, zc = host["row_argmax"][a:b], host["row_zmax"][a:b], host["row_zchild"][a:b]
        dz = np.abs(zm - res.row_zmax)
        assert np.all(dz <= H.LOGIT_TOL), f"seq{i}: zmax off by {dz.max():.4f} at row {int(dz.argmax())}"
        assert np.isnan(zc[0])
        for j in range(1, n):
            ref = res.logits[par[j], int(tokens[j])]
            assert abs(zc[j] - ref) <= H.LOGIT_TOL, f"seq{i}: zchild row {j} off by {abs(zc[j] - ref):.4f}"
            stats["max_dz"] = max(stats["max_dz"], float(abs(zc[j] - ref)))
        stats["max_dz"] = max(stats["max_dz"], float(dz.max()))
        for j in range(n):
            if res.row_gap[j] > H.GAP_EXACT:
                assert am[j] == res.row_argmax[j], f"seq{i}: row {j} argmax"
        # the library's path follows from its own rows
        g_acc = int(host["accept_len"][i])
        g_path = host["accept_rows"][i][:g_acc].tolist()
        g_emit = host["emit_tokens"][i][:g_acc + 1].tolist()
        assert int(host["n_emit"][i]) == g_acc + 1
        want_path, want_emit = traverse_rows(par, tokens, am, zm, zc, log_tau)
        assert g_path == want_path and g_emit == want_emit, f"seq{i}: path {g_path} vs own rows {want_path}"
        clear = oracle_decisive_steps(res, par, tokens, log_tau)
        m = min(clear, len(res.path))
        assert g_path[:m] == list(res.path)[:m], f"seq{i}: path leaves the oracle's inside its clear part"
        stats["clear_moves"] = stats.get("clear_moves", 0) + m
        if clear == len(res.path) + 1:
            assert g_path == list(res.path) and g_emit == list(res.emitted), f"seq{i}: path differs from the oracle's"
            stats["exact"] += 1
        else:
            stats["tolerated"] += 1
    if not second_step:
        return stats, host, res_l
    # ---- KV maintenance with the ORACLE's path on both sides, then a plain chain step on top of it
    acc = np.asarray([r.accept_len for r in res_l], np.int32)
    rows = np.zeros((S, max_q), np.int32)
    for i, r in enumerate(res_l):
        rows[i, :r.accept_len] = r.path
    before = kv.seq_lens.cpu().numpy().copy()
    eng.commit_tree(eng._i32(acc), eng._i32(rows))
    torch.cuda.synchronize()
    assert (kv.seq_lens.cpu().numpy() - before).tolist() == (acc + 1).tolist()
    pend2, drafts2, res2 = [], [], []
    for i, r in enumerate(res_l):
        caches[i].commit([0] + list(r.path))
        p2 = int(r.emitted[-1])
        g2 = O.greedy_continuation(caches[i], p2, 6)
        d2 = I.plant_draft(g2, 6, (i * 3) % 7, wl.seqs[i].rand_tokens, cfg.vocab, False)
        pend2.append(p2); drafts2.append(d2)
        res2.append(O.verify_cached(caches[i], p2, d2, keep_logits=True))
    toks2, cu2 = I.pack_queries(pend2, drafts2)
    out2 = eng.verify_regions(eng._i32(toks2), eng._i32(cu2), 7, 7 * S)
    eng.check_device("second step")
    torch.cuda.synchronize()
    h2 = {n: t.cpu().numpy() for n, t in out2.items()}
    st2 = {}
    for i in range(S):
        a, b = int(cu2[i]), int(cu2[i + 1])
        H.compare_rows(f"seq{i} step2", res2[i], drafts2[i], h2["row_argmax"][a:b], h2["row_zmax"][a:b],
                       h2["row_zdraft"][a:b], st2)
        H.compare_sequence(f"seq{i} step2", res2[i], drafts2[i], h2["accept_len"][i], h2["emit_tokens"][i],
                           h2["n_emit"][i], h2["row_argmax"][a:b], st2)
    stats["step2_max_dz"] = st2["max_dz"]
    return stats, host, res_l


@pytest.mark.parametrize("log_tau", [0.0, LOG_TAU_PAPER], ids=["greedy", "tau0.75"])
def test_tiny_trees_match_oracle(log_tau):
    wl = I.tiny_workload(n_regions=5, draft_len=40)
    stats, _, _ = run_tree_case(wl, [40, 17, 1, 0, 127], log_tau)
    assert stats["exact"] + stats["tolerated"] == 5 and stats["exact"] >= 1
    print("tiny trees", log_tau, stats)


@pytest.mark.parametrize("log_tau", [0.0, LOG_TAU_PAPER], ids=["greedy", "tau0.75"])
def test_small_decoder_trees_match_oracle(log_tau):
    """Layer shape of the 24-layer decoder (GQA 16/8: 64 tokens per q-tile, so 127-node trees span two q-tiles and
    their ancestry masks cross KV tiles), 2 layers, prefixes that end inside a KV block."""
    wl = I.region_workload(seed=91, n_regions=4, prefix_lo=70, prefix_hi=300, draft_mean=60, draft_lo=8, draft_hi=120,
                           cfg=I.small_decoder(2, 8192), name="small_trees")
    stats, _, _ = run_tree_case(wl, [127, 64, 90, 33], log_tau)
    assert stats["exact"] + stats["tolerated"] == 4 and stats["clear_moves"] >= 4
    print("small trees", log_tau, stats)


def test_many_short_trees_in_one_call():
    """Forty sequences with trees of 0 to 59 nodes in one call (more sequences than any grid dimension the other cases
    reach), then the compacting commit and a chain step on top."""
    wl = I.tiny_workload(n_regions=40, draft_len=30, prefix_len=96, n_visual=32)
    rng = np.random.default_rng(1)
    nodes = [int(x) for x in rng.integers(0, 60, size=40)]
    stats, _, _ = run_tree_case(wl, nodes, LOG_TAU_PAPER)
    assert stats["exact"] + stats["tolerated"] == 40 and stats["max_dz"] < H.LOGIT_TOL


def test_a_chain_given_as_a_tree_equals_the_chain_call():
    """parent[j] = j - 1 is the linear draft: same integers as hsd_verify_regions, same logits."""
    from paper_2602_12957_b200 import binding as B
    wl = I.tiny_workload(n_regions=3, draft_len=20)
    _, host, _ = run_tree_case(wl, [20, 20, 20], 0.0, flags=B.HSD_FLAG_DETERMINISTIC, second_step=False, chain=True)
    weights = I.make_weights(wl.cfg, wl.seed)
    orc = H.oracle_regions(wl, weights, np.float64)          # plants the same drafts from the same greedy paths
    per, _, (toks, cu, total_q) = H.gpu_regions(wl, weights, {i: o.pending for i, o in orc.items()},
                                                {i: o.draft for i, o in orc.items()}, B.HSD_FLAG_DETERMINISTIC)
    for i in range(3):
        a = int(per[i]["accept_len"])
        assert int(host["accept_len"][i]) == a
        assert host["emit_tokens"][i][:a + 1].tolist() == per[i]["emit"][:a + 1].tolist()
        assert host["accept_rows"][i][:a].tolist() == list(range(1, a + 1))
        lo, hi = int(cu[i]), int(cu[i + 1])
        assert np.array_equal(host["row_argmax"][lo:hi], per[i]["row_argmax"])
        assert np.allclose(host["row_zmax"][lo:hi], per[i]["row_zmax"], rtol=0, atol=1e-5)
        assert np.allclose(host["row_zchild"][lo + 1:hi], per[i]["row_zdraft"][:-1], rtol=0, atol=1e-5)


def test_tree_argument_and_device_checks():
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    wl = I.tiny_workload(n_regions=2, draft_len=8)
    weights = I.make_weights(wl.cfg, wl.seed)
    model = R.DeviceModel(wl.cfg, weights, 0)
    kv = R.KvCache(model, [400, 400], seed=1)
    eng = R.Engine(model, kv, 600, 2)
    eng.prefill([s.prefix_embeds for s in wl.seqs], [s.prefix_ids for s in wl.seqs])
    toks = eng._i32(np.arange(10) % 7)
    cu = eng._i32([0, 5, 10])
    good = np.asarray([-1, 0, 0, 1, 2, -1, 0, 1, 1, 3], np.int32)
    out = eng.verify_tree(toks, cu, eng._i32(good), 5, 10)
    eng.check_device("good tree")
    # more rows per sequence than a tree may have: refused on the host
    st = B.hsd_verify_tree(model.ctx, kv.c, 2, cu, toks, eng._i32(good), None, 129, 300, 0.0, out["accept_len"],
                           out["emit_tokens"], out["n_emit"], out["accept_rows"], None, None, None, eng.ws.ptr,
                           eng.ws.bytes, torch.cuda.current_stream().cuda_stream)
    assert st == B.HSD_ERR_TOO_LONG
    # a workspace sized for total_q rows only is too small
    small = R.Workspace(model, 10, 2)
    st = B.hsd_verify_tree(model.ctx, kv.c, 2, cu, toks, eng._i32(good), None, 5, 10, 0.0, out["accept_len"],
                           out["emit_tokens"], out["n_emit"], out["accept_rows"], None, None, None, small.ptr,
                           small.bytes, torch.cuda.current_stream().cuda_stream)
    assert st == B.HSD_ERR_WORKSPACE
    # a parent that is not an earlier row: device status 7 with the packed row, no decision (-1, nothing emitted), context usable
    for bad_row, bad_val in ((3, 3), (7, 9), (5, 0), (2, -1)):
        bad = good.copy()
        bad[bad_row] = bad_val
        out["accept_len"].fill_(-5)
        eng.verify_tree(toks, cu, eng._i32(bad), 5, 10, out=out)
        st, words = eng.device_status()
        assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 7, (bad_row, words)
        assert out["accept_len"].cpu().tolist() == [-1, -1] and out["n_emit"].cpu().tolist() == [0, 0]
    eng.verify_tree(toks, cu, eng._i32(good), 5, 10, out=out)
    eng.check_device("after the bad trees")
    assert all(0 <= a <= 4 for a in out["accept_len"].cpu().tolist())


def test_head_dim_128_trees_match_oracle_and_compact():
    """Head dimension 128 through the tree path: ancestry masks, traversal at tau 0.75, compaction of 256-byte KV rows,
    then a chain step on top of the compacted cache."""
    cfg = I.ModelConfig(n_layers=2, d_model=1024, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=4096, vocab=8192)
    wl = I.region_workload(seed=92, n_regions=4, prefix_lo=70, prefix_hi=300, draft_mean=60, draft_lo=8, draft_hi=120,
                           cfg=cfg, name="hd128_trees")
    stats, _, _ = run_tree_case(wl, [127, 64, 90, 33], LOG_TAU_PAPER)
    assert stats["exact"] + stats["tolerated"] == 4 and stats["max_dz"] < H.LOGIT_TOL
    print("hd128 trees", stats)
