"""GPU parity of the page-level stage: one sequence, a long draft verified chunk by chunk through hsd_verify_page
with KV commit / rollback after every chunk, against the CPU oracle run in lock-step."""
import numpy as np
import pytest

from oracle import hsd_oracle as O
from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def _page_schedule(cfg, seed, n_visual, n_prompt, draft_len, chunk_len, log_tau=0.0, attn_plan=None, n_err=3):
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    wl = I.page_workload(seed=seed, n_visual=n_visual, n_prompt=n_prompt, draft_len=draft_len, chunk_len=chunk_len, cfg=cfg)
    s = wl.seqs[0]
    weights = I.make_weights(cfg, wl.seed)
    model = O.Decoder(cfg, weights, np.float64)
    cache = O.CachedSequence(model)
    pending = cache.prefill(s.prefix_embeds, s.prefix_ids)
    greedy = O.greedy_continuation(cache, pending, draft_len)
    # page draft = the oracle's greedy path with a few substitution errors (the draft re-aligns after each)
    rng = np.random.default_rng(seed)
    draft = np.asarray(greedy, np.int32).copy()
    for pos in sorted(rng.choice(draft_len, size=n_err, replace=False)):
        draft[pos] = (draft[pos] + 1 + int(rng.integers(0, cfg.vocab - 1))) % cfg.vocab
    dm = R.DeviceModel(cfg, weights, 0)
    if attn_plan is not None:
        B.check(B.hsd_debug_set_attn_plan(dm.ctx, attn_plan[0], attn_plan[1]))
    kv = R.KvCache(dm, [s.prefix_len + draft_len + chunk_len + 2], seed=seed, poison=True)
    eng = R.Engine(dm, kv, max(s.prefix_len, chunk_len + 1), 1)
    first = eng.prefill([s.prefix_embeds], [s.prefix_ids])
    eng.check_device("prefill")
    pl = np.sort(cache.last_prefill_logits)
    if pl[-1] - pl[-2] > H.GAP_EXACT:
        assert int(first[0].item()) == pending
    stats, start, n_chunks = {}, 0, 0
    pend_dev = torch.tensor([pending], dtype=torch.int32, device=eng.dev)
    while start < draft_len:
        chunk = draft[start:start + chunk_len]
        res = O.verify_cached(cache, pending, chunk, log_tau=log_tau, keep_logits=True)
        out = eng.verify_page(0, pend_dev, eng._i32(chunk), log_tau=log_tau)
        eng.check_device("verify_page")
        g = {k: v.cpu().numpy() for k, v in out.items()}
        k = len(chunk)
        H.compare_rows(f"chunk@{start}", res, chunk, g["row_argmax"][:k + 1], g["row_zmax"][:k + 1], g["row_zdraft"][:k + 1], stats)
        if log_tau == 0.0:
            H.compare_sequence(f"chunk@{start}", res, chunk, g["accept_len"][0], g["emit_tokens"][0], g["n_emit"][0],
                               g["row_argmax"][:k + 1], stats)
        else:   # thresholded rule: decisive wherever the test's margin is clear of the logit tolerance
            a = int(g["accept_len"][0])
            margin = (res.row_zdraft[:k] - res.row_zmax[:k]) - log_tau
            if np.all(np.abs(margin[:min(res.accept_len + 1, k)]) > 2 * H.LOGIT_TOL):
                assert a == res.accept_len
        # keep both sides in lock-step on the oracle's decision (KV commit with a caller-chosen length)
        acc = torch.tensor([res.accept_len], dtype=torch.int32, device=eng.dev)
        eng.commit(acc)
        pending = O.commit_step(cache, res)
        pend_dev = torch.tensor([pending], dtype=torch.int32, device=eng.dev)
        assert int(kv.seq_lens[0].item()) == cache.length
        start += res.accept_len + 1
        n_chunks += 1
    return stats, n_chunks


def test_page_chunks_with_commit_and_rollback_match_oracle():
    cfg = I.small_decoder(2, 8192)
    stats, n_chunks = _page_schedule(cfg, seed=31, n_visual=200, n_prompt=40, draft_len=300, chunk_len=96)
    print("page", stats, n_chunks)
    assert n_chunks >= 4 and stats["max_dz"] < H.LOGIT_TOL


def test_page_chunk_over_long_context_with_kv_slices():
    """A context of ~17 KV tiles cut into slices (the batch-1 page regime, where slicing is what fills the GPU)."""
    cfg = I.small_decoder(1, 4096)
    stats, n_chunks = _page_schedule(cfg, seed=32, n_visual=1000, n_prompt=24, draft_len=130, chunk_len=129,
                                     attn_plan=(1 << 20, 2), n_err=1)
    print("long", stats, n_chunks)
    assert stats["max_dz"] < H.LOGIT_TOL


def test_thresholded_acceptance_matches_eq11_on_raw_logits():
    cfg = I.small_decoder(1, 4096)
    stats, n_chunks = _page_schedule(cfg, seed=33, n_visual=90, n_prompt=10, draft_len=120, chunk_len=60,
                                     log_tau=float(np.log(0.75)), n_err=4)
    print("tau", stats, n_chunks)
    assert stats["max_dz"] < H.LOGIT_TOL


def test_empty_draft_is_a_plain_decode_step():
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = I.TINY
    wl = I.tiny_workload()
    weights = I.make_weights(cfg, wl.seed)
    s = wl.seqs[0]
    model = O.Decoder(cfg, weights, np.float64)
    cache = O.CachedSequence(model)
    pending = cache.prefill(s.prefix_embeds, s.prefix_ids)
    res = O.verify_cached(cache, pending, np.zeros(0, np.int64), keep_logits=True)
    dm = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(dm, [s.prefix_len + 4], seed=3)
    eng = R.Engine(dm, kv, s.prefix_len, 1)
    eng.prefill([s.prefix_embeds], [s.prefix_ids])
    out = eng.verify_page(0, torch.tensor([pending], dtype=torch.int32, device=eng.dev),
                          torch.zeros(0, dtype=torch.int32, device=eng.dev))
    eng.check_device("verify_page")
    assert int(out["accept_len"][0]) == 0 and int(out["n_emit"][0]) == 1
    assert abs(float(out["row_zmax"][0]) - res.row_zmax[0]) < H.LOGIT_TOL
    if res.row_gap[0] > H.GAP_EXACT:
        assert int(out["emit_tokens"][0, 0]) == res.emitted[0]


def test_head_dim_128_page_chunks_with_commit_and_rollback_match_oracle():
    cfg = I.ModelConfig(n_layers=2, d_model=1024, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=4096, vocab=8192)
    stats, n_chunks = _page_schedule(cfg, seed=34, n_visual=200, n_prompt=40, draft_len=300, chunk_len=96)
    print("hd128 page", stats, n_chunks)
    assert n_chunks >= 4 and stats["max_dz"] < H.LOGIT_TOL
