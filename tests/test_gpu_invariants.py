"""GPU-only invariants of the paged, varlen step (run with the deterministic flag, so equality is bit-exact):
physical block placement, batch composition and order must not change a sequence's results; device-side checks
turn bad inputs into status codes instead of faults."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def _run(wl, weights, pend, drafts, seed, order):
    from paper_2602_12957_b200 import binding as B
    per, eng, _ = H.gpu_regions(wl, weights, pend, drafts, B.HSD_FLAG_DETERMINISTIC, seed=seed, order=order)
    return per


def test_block_placement_batch_order_and_batch_membership_do_not_change_results():
    cfg = I.small_decoder(1, 4096)
    # prefix lengths that end exactly on / just around a 64-token block boundary, drafts crossing 1-3 blocks
    wl = I.region_workload(seed=5, n_regions=5, prefix_lo=60, prefix_hi=200, draft_mean=40, draft_lo=5, draft_hi=140, cfg=cfg)
    for s, L in zip(wl.seqs, (64, 128, 127, 65, 190)):
        s.prefix_embeds = s.prefix_embeds[:L] if s.prefix_len >= L else np.concatenate([s.prefix_embeds] * 4)[:L]
        s.prefix_ids = np.full(L, -1, np.int32)
    weights = I.make_weights(cfg, 11)
    rng = np.random.default_rng(0)
    pend = {i: int(rng.integers(0, cfg.vocab)) for i in range(5)}
    drafts = {i: wl.seqs[i].rand_tokens[:wl.seqs[i].draft_len] for i in range(5)}
    base = _run(wl, weights, pend, drafts, seed=0, order=None)
    perm = _run(wl, weights, pend, drafts, seed=123, order=None)            # other physical blocks
    rev = _run(wl, weights, pend, drafts, seed=7, order=[4, 2, 0, 3, 1])    # other batch order
    sub = _run(wl, weights, {i: pend[i] for i in (1, 3)}, {i: drafts[i] for i in (1, 3)}, seed=9, order=None)
    for other, ids in ((perm, range(5)), (rev, range(5)), (sub, (1, 3))):
        for i in ids:
            for key in ("row_argmax", "row_zmax", "accept_len", "n_emit", "first_token"):
                assert np.array_equal(np.asarray(base[i][key]), np.asarray(other[i][key])), (i, key)
            k = len(drafts[i])
            assert np.array_equal(base[i]["row_zdraft"][:k], other[i]["row_zdraft"][:k])


def test_two_runs_are_bit_identical():
    cfg = I.small_decoder(2, 8192)
    wl = I.region_workload(seed=6, n_regions=6, prefix_lo=100, prefix_hi=700, draft_mean=60, draft_lo=8, draft_hi=200, cfg=cfg)
    weights = I.make_weights(cfg, 12)
    pend = {i: 17 + i for i in range(6)}
    drafts = {i: wl.seqs[i].rand_tokens[:wl.seqs[i].draft_len] for i in range(6)}
    a = _run(wl, weights, pend, drafts, seed=1, order=None)
    b = _run(wl, weights, pend, drafts, seed=1, order=None)
    for i in range(6):
        assert np.array_equal(a[i]["row_zmax"], b[i]["row_zmax"]) and np.array_equal(a[i]["row_argmax"], b[i]["row_argmax"])


def test_device_side_checks_report_instead_of_faulting():
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = I.TINY
    wl = I.tiny_workload()
    weights = I.make_weights(cfg, wl.seed)
    dm = R.DeviceModel(cfg, weights, 0)
    S = 2
    kv = R.KvCache(dm, [200, 200], seed=0)
    eng = R.Engine(dm, kv, 256, S)
    eng.prefill([s.prefix_embeds for s in wl.seqs[:S]], [s.prefix_ids for s in wl.seqs[:S]])
    eng.check_device("prefill")
    lens0 = kv.seq_lens.clone()
    toks = np.array([1, 2, 3, 4, 5, 6], np.int32)
    cu = np.array([0, 3, 6], np.int32)

    def call(t, c, max_q, total):
        out = eng.verify_regions(eng._i32(t), eng._i32(c), max_q, total)
        torch.cuda.synchronize()
        return eng.device_status(), out

    (st, words), _ = call(toks, cu, 3, 6)
    assert st == B.HSD_OK
    bad = toks.copy(); bad[4] = cfg.vocab + 5                     # token id out of range
    (st, words), _ = call(bad, cu, 3, 6)
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 3 and words[1] == 4
    (st, words), _ = call(toks, np.array([0, 4, 3], np.int32), 4, 6)   # offsets not monotone
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 1
    (st, words), _ = call(toks, np.array([0, 5, 6], np.int32), 3, 6)   # a sequence longer than max_q_len
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 2
    kv.seq_lens[1] = kv.max_blocks * 64 - 1                      # one free row left, three needed
    (st, words), _ = call(toks, cu, 3, 6)
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 4 and words[1] == 1
    kv.seq_lens.copy_(lens0)
    (st, words), _ = call(toks, cu, 3, 6)                         # and the context is still usable afterwards
    assert st == B.HSD_OK
    # host-side refusals: nothing is launched
    n0 = B.hsd_launch_count(dm.ctx)
    o = eng.alloc_outputs(S, 3, 6)
    args = (dm.ctx, kv.c, S, eng._i32(cu), eng._i32(toks), None)
    tail = (o["accept_len"], o["emit_tokens"], o["n_emit"], o["row_argmax"], o["row_zmax"], o["row_zdraft"])
    st_ = torch.cuda.current_stream().cuda_stream
    assert B.hsd_verify_regions(*args, 3, 6, 0.0, *tail, eng.ws.ptr, 1024, st_) == B.HSD_ERR_WORKSPACE
    assert B.hsd_verify_regions(*args, 3, 6, 0.0, *tail, eng.ws.ptr + 8, eng.ws.bytes, st_) == B.HSD_ERR_WORKSPACE
    assert B.hsd_verify_regions(*args, B.HSD_MAX_Q_LEN + 1, B.HSD_MAX_Q_LEN + 5, 0.0, *tail, eng.ws.ptr, eng.ws.bytes, st_) == B.HSD_ERR_TOO_LONG
    assert B.hsd_verify_regions(*args, 3, 6, 0.5, *tail, eng.ws.ptr, eng.ws.bytes, st_) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_verify_regions(*args, 3, 6, 0.0, None, *tail[1:], eng.ws.ptr, eng.ws.bytes, st_) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_launch_count(dm.ctx) == n0


def test_failed_device_check_leaves_cache_and_lengths_untouched():
    """A step that trips a device-side check is a no-op: no K/V row is written, no length advances, and the decision
    outputs say so (accept_len -1, n_emit 0) — also on a workspace no valid call has ever filled (zeroed here, so that
    a store through a never-written row index would land in bounds, on physical row 0, and show up in the comparison)."""
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = I.TINY
    wl = I.tiny_workload()
    weights = I.make_weights(cfg, wl.seed)
    dm = R.DeviceModel(cfg, weights, 0)
    S = 2
    kv = R.KvCache(dm, [320, 320], seed=0)
    eng = R.Engine(dm, kv, 512, S)
    eng.prefill([s.prefix_embeds for s in wl.seqs[:S]], [s.prefix_ids for s in wl.seqs[:S]])
    eng.check_device("prefill")
    torch.cuda.synchronize()
    k0, v0, lens0 = kv.k_pool.clone(), kv.v_pool.clone(), kv.seq_lens.clone()
    toks = np.array([1, 2, 3, 4, 5, 6], np.int32)
    cu = np.array([0, 3, 6], np.int32)
    bad_tok = toks.copy(); bad_tok[4] = cfg.vocab + 5
    cases = [("token", bad_tok, cu, 3, 3), ("offsets", toks, np.array([0, 4, 3], np.int32), 4, 1),
             ("too_long", toks, np.array([0, 5, 6], np.int32), 3, 2)]

    def fresh_engine():
        e = R.Engine(dm, kv, 512, S)
        e.ws._raw.zero_()
        return e

    def unchanged():
        torch.cuda.synchronize()
        return (torch.equal(kv.k_pool, k0) and torch.equal(kv.v_pool, v0) and torch.equal(kv.seq_lens, lens0))

    for name, t, c, max_q, code in cases:
        e2 = fresh_engine()
        out = e2.alloc_outputs(S, max_q, 6)
        for v in out.values():
            v.fill_(7)
        out = e2.verify_regions(e2._i32(t), e2._i32(c), max_q, 6, out=out)
        e2.commit(out["accept_len"])
        st, words = e2.device_status()
        assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == code, (name, st, words)
        assert out["accept_len"].cpu().tolist() == [-1, -1] and out["n_emit"].cpu().tolist() == [0, 0], name
        assert unchanged(), name
    # capacity: one free row left, three needed (lengths are the caller's; restored afterwards)
    e2 = fresh_engine()
    kv.seq_lens[1] = kv.max_blocks * 64 - 1
    lens_cap = kv.seq_lens.clone()
    out = e2.verify_regions(e2._i32(toks), e2._i32(cu), 3, 6)
    e2.commit(out["accept_len"])
    st, words = e2.device_status()
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 4
    assert torch.equal(kv.seq_lens, lens_cap) and torch.equal(kv.k_pool, k0) and torch.equal(kv.v_pool, v0)
    kv.seq_lens.copy_(lens0)
    # the host-buffer entry with commit folded in: the error comes back and nothing moved
    e2 = fresh_engine()
    h_t, h_c = torch.from_numpy(bad_tok).pin_memory(), torch.from_numpy(cu).pin_memory()
    h_acc = torch.full((S,), 7, dtype=torch.int32).pin_memory()
    h_nem = torch.full((S,), 7, dtype=torch.int32).pin_memory()
    h_emit = torch.full((S, 3), 7, dtype=torch.int32).pin_memory()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):          # eager, capturing and replayed calls of the library's own graph
        rc, _ = B.hsd_verify_regions_host(dm.ctx, kv.c, S, h_c, h_t, None, 0.0, 1, h_acc, h_emit, h_nem, e2.ws.ptr,
                                          e2.ws.bytes, side.cuda_stream)
        assert rc == B.HSD_ERR_DEVICE_CHECK
        assert h_acc.tolist() == [-1, -1] and h_nem.tolist() == [0, 0]
        assert unchanged()
    # candidate trees: a parent pointer that names a later row
    e2 = R.Engine(dm, kv, 512, S)
    e2.ws._raw.zero_()
    parent = np.array([-1, 0, 1, -1, 2, 0], np.int32)          # row 1 of the second tree points at row 2
    out = e2.verify_tree(e2._i32(toks), e2._i32(cu), e2._i32(parent), 3, 6)
    e2.commit_tree(out["accept_len"], out["accept_rows"])
    st, words = e2.device_status()
    assert st == B.HSD_ERR_DEVICE_CHECK and words[0] == 7
    assert out["accept_len"].cpu().tolist() == [-1, -1]
    assert unchanged()
    # and the context still works
    out = eng.verify_regions(eng._i32(toks), eng._i32(cu), 3, 6)
    st, _ = eng.device_status()
    assert st == B.HSD_OK and min(out["accept_len"].cpu().tolist()) >= 0
