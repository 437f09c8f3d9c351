"""GPU parity: whole verify step through the C-ABI against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def run_region_parity(wl, flags=0, dtype=np.float64, which=None, attn_plan=None):
    weights = I.make_weights(wl.cfg, wl.seed)
    orc = H.oracle_regions(wl, weights, dtype, which)
    per, eng, _ = H.gpu_regions(wl, weights, {i: o.pending for i, o in orc.items()},
                                {i: o.draft for i, o in orc.items()}, flags, attn_plan=attn_plan)
    stats = {}
    for i, o in orc.items():
        g = per[i]
        H.check_first_token(f"seq{i}", o, g["first_token"])
        H.compare_rows(f"seq{i}", o.res, o.draft, g["row_argmax"], g["row_zmax"], g["row_zdraft"], stats)
        H.compare_sequence(f"seq{i}", o.res, o.draft, g["accept_len"], g["emit"], g["n_emit"], g["row_argmax"], stats)
    return stats, orc, per, eng


@pytest.mark.parametrize("flags", [1, 2, 0], ids=["simt", "simt_attention", "tensor"])
def test_tiny_config_matches_oracle(flags):
    stats, orc, per, _ = run_region_parity(I.tiny_workload(), flags)
    assert stats["exact_rows"] + stats["near_tie_rows"] == 4 * 17
    assert stats["max_dz"] < H.LOGIT_TOL
    print("tiny", flags, stats)


@pytest.mark.parametrize("flags", [1, 0], ids=["simt", "tensor"])
def test_qk_norm_decoder_matches_oracle(flags):
    """Per-head RMSNorm of q and k before the rotary embedding (the Qwen3-style decoder variant): the Tiny shape and
    a GQA shape with several q-tiles, through the fused QKV epilogue and through the plain kernels."""
    import dataclasses
    tiny = dataclasses.replace(I.TINY, qk_norm=True)
    stats, _, _, _ = run_region_parity(I.tiny_workload(cfg=tiny), flags)
    assert stats["max_dz"] < H.LOGIT_TOL
    cfg = dataclasses.replace(I.small_decoder(2, 8192), qk_norm=True)
    wl = I.region_workload(seed=78, n_regions=3, prefix_lo=70, prefix_hi=200, draft_mean=50, draft_lo=8, draft_hi=150,
                           cfg=cfg, name="small_regions_qk_norm")
    stats2, _, _, _ = run_region_parity(wl, flags)
    assert stats2["max_dz"] < H.LOGIT_TOL
    # the norm is really applied: the same weights without it give other logits
    plain = run_region_parity(I.tiny_workload(), flags)[2]
    with_norm = run_region_parity(I.tiny_workload(cfg=tiny), flags)[2]
    assert np.max(np.abs(plain[0]["row_zmax"] - with_norm[0]["row_zmax"])) > 1e-2
    print("qk_norm", flags, stats, stats2)


@pytest.mark.parametrize("flags", [2, 0], ids=["simt_attention", "tensor"])
def test_small_decoder_regions_match_oracle(flags):
    """Same layer shape as the 24-layer decoder (GQA 16/8, d 1024, FFN 4096), 2 layers, vocab 8192: several
    q-tiles per sequence, ragged tails, prefixes that end inside a KV block."""
    wl = I.region_workload(seed=77, n_regions=5, prefix_lo=70, prefix_hi=330, draft_mean=60, draft_lo=8, draft_hi=200,
                           cfg=I.small_decoder(2, 8192), name="small_regions")
    stats, orc, per, _ = run_region_parity(wl, flags)
    print("small", flags, stats, [(len(o.draft), o.res.accept_len) for o in orc.values()])
    assert stats["max_dz"] < H.LOGIT_TOL


@pytest.mark.parametrize("plan", [(1 << 20, 1), (1, 1 << 20)], ids=["max_slices", "no_slices"])
def test_attention_kv_slicing_does_not_change_the_result(plan):
    """The KV range of a query tile cut into as many slices as allowed (partials combined by the last slice to
    finish) and not cut at all: both within the oracle's tolerance, on contexts of 2 to 9 KV tiles."""
    wl = I.region_workload(seed=78, n_regions=4, prefix_lo=100, prefix_hi=520, draft_mean=50, draft_lo=8, draft_hi=150,
                           cfg=I.small_decoder(2, 8192), name="small_regions_slicing")
    stats, orc, per, _ = run_region_parity(wl, 0, attn_plan=plan)
    print("slicing", plan, stats)
    assert stats["max_dz"] < H.LOGIT_TOL


def test_one_verify_call_equals_sequential_single_token_steps_on_gpu():
    """The library against itself: k+1 plain decode steps (empty drafts, commit each) must reproduce the rows of
    one verify call over the tokens they emitted — same kernels, same K/V rows, same tile boundaries."""
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = I.small_decoder(2, 8192)
    wl = I.region_workload(seed=91, n_regions=3, prefix_lo=60, prefix_hi=200, draft_mean=40, draft_lo=20, draft_hi=70,
                           cfg=cfg)
    weights = I.make_weights(cfg, 5)
    model = R.DeviceModel(cfg, weights, B.HSD_FLAG_DETERMINISTIC)   # bit-equality needs a fixed summation order
    S = len(wl.seqs)
    k = 20
    kv = R.KvCache(model, [s.prefix_len + k + 2 for s in wl.seqs], seed=1)
    eng = R.Engine(model, kv, max(sum(s.prefix_len for s in wl.seqs), S * (k + 1)), S)
    first = eng.prefill([s.prefix_embeds for s in wl.seqs], [s.prefix_ids for s in wl.seqs])
    base = kv.seq_lens.clone()
    cu1 = eng._i32(np.arange(S + 1))
    pending, toks, zs = first.clone(), [], []
    for _ in range(k + 1):
        o = eng.verify_regions(pending, cu1, 1, S)
        eng.commit(o["accept_len"])
        zs.append(o["row_zmax"].clone())
        pending = o["emit_tokens"][:, 0].clone()
        toks.append(pending)
    seq_z = torch.stack(zs, 1).cpu().numpy()              # [S, k+1]
    greedy = torch.stack(toks, 1).cpu().numpy()           # [S, k+1]
    assert (kv.seq_lens - base).cpu().numpy().tolist() == [k + 1] * S
    kv.seq_lens.copy_(base)
    q, cu = I.pack_queries(first.cpu().numpy(), [greedy[i, :k] for i in range(S)])
    o = eng.verify_regions(eng._i32(q), eng._i32(cu), k + 1, S * (k + 1))
    eng.check_device("verify")
    z = o["row_zmax"].cpu().numpy().reshape(S, k + 1)
    am = o["row_argmax"].cpu().numpy().reshape(S, k + 1)
    assert np.array_equal(am, greedy), "teacher-forced rows must reproduce the sequential greedy tokens"
    assert np.array_equal(z, seq_z), f"max |dz| {np.abs(z - seq_z).max()}"
    assert o["accept_len"].cpu().numpy().tolist() == [k] * S


def test_host_buffer_call_replays_a_captured_graph_with_fresh_inputs():
    """On a side stream the host-buffer entry captures the step into a CUDA graph at the second call of one shape and
    replays it afterwards.  Every call (eager, capturing, replayed) must give the integers of the plain device call,
    also when the token values (hence accept lengths) change between calls, and account the same number of launches."""
    import torch
    from paper_2602_12957_b200 import binding as B
    wl = I.tiny_workload()
    weights = I.make_weights(wl.cfg, wl.seed)
    orc = H.oracle_regions(wl, weights, np.float64)
    per, eng, (toks, cu, total_q) = H.gpu_regions(wl, weights, {i: o.pending for i, o in orc.items()},
                                                  {i: o.draft for i, o in orc.items()}, B.HSD_FLAG_DETERMINISTIC)
    S = len(orc)
    ctx = eng.model.ctx
    max_q = int(np.diff(cu).max())
    lens0 = eng.kv.seq_lens.clone()
    side = torch.cuda.Stream()
    rng = np.random.default_rng(11)
    variants = [toks.copy()]
    for _ in range(3):                                   # same shape, other draft tokens after the pending one
        v = toks.copy()
        for i in range(S):
            lo, hi = int(cu[i]) + 1, int(cu[i + 1])
            if hi > lo:
                cut = int(rng.integers(lo, hi))
                v[cut:hi] = rng.integers(0, wl.cfg.vocab, hi - cut)
        variants.append(v)
    variants.append(toks.copy())
    h_cu = torch.from_numpy(cu).pin_memory()
    counts = []
    for v in variants:
        # plain device call on the same inputs (no commit), as the expected integers
        d_t, d_c = eng._i32(v), eng._i32(cu)
        out = eng.verify_regions(d_t, d_c, max_q, total_q)
        torch.cuda.synchronize()
        exp_acc = out["accept_len"].cpu().numpy()
        exp_emit = out["emit_tokens"].cpu().numpy().reshape(S, -1)
        h_toks = torch.from_numpy(v).pin_memory()
        h_acc = torch.full((S,), -7, dtype=torch.int32).pin_memory()
        h_nem = torch.full((S,), -7, dtype=torch.int32).pin_memory()
        h_emit = torch.full((S, max_q), -7, dtype=torch.int32).pin_memory()
        n0 = B.hsd_launch_count(ctx)
        rc, mq = B.hsd_verify_regions_host(ctx, eng.kv.c, S, h_cu, h_toks, None, 0.0, 1, h_acc, h_emit, h_nem,
                                           eng.ws.ptr, eng.ws.bytes, side.cuda_stream)
        B.check(rc, "hsd_verify_regions_host")
        counts.append(B.hsd_launch_count(ctx) - n0)
        assert mq == max_q
        assert h_acc.numpy().tolist() == exp_acc.tolist()
        assert h_nem.numpy().tolist() == (exp_acc + 1).tolist()
        for j in range(S):
            a = int(exp_acc[j])
            assert h_emit[j, :a + 1].tolist() == exp_emit[j, :a + 1].tolist()
        assert (eng.kv.seq_lens - lens0).cpu().numpy().tolist() == (exp_acc + 1).tolist()   # the commit ran
        eng.kv.seq_lens.copy_(lens0)
        torch.cuda.synchronize()
    assert len(set(counts)) == 1 and counts[0] > 0, counts


def test_host_buffer_call_matches_the_device_call_and_commits():
    """hsd_verify_regions_host (host buffers in, host buffers out, commit folded in) against hsd_verify_regions +
    hsd_kv_commit on the same inputs: identical integers, and the committed lengths advance by accept_len + 1."""
    import torch
    from paper_2602_12957_b200 import binding as B
    wl = I.tiny_workload()
    weights = I.make_weights(wl.cfg, wl.seed)
    orc = H.oracle_regions(wl, weights, np.float64)
    per, eng, (toks, cu, total_q) = H.gpu_regions(wl, weights, {i: o.pending for i, o in orc.items()},
                                                  {i: o.draft for i, o in orc.items()}, B.HSD_FLAG_DETERMINISTIC)
    S = len(orc)
    before = eng.kv.seq_lens.cpu().numpy().copy()
    h_toks, h_cu = torch.from_numpy(toks).pin_memory(), torch.from_numpy(cu).pin_memory()
    max_q = int(np.diff(cu).max())
    h_acc = torch.full((S,), -7, dtype=torch.int32).pin_memory()
    h_nem = torch.full((S,), -7, dtype=torch.int32).pin_memory()
    h_emit = torch.full((S, max_q), -7, dtype=torch.int32).pin_memory()
    rc, mq = B.hsd_verify_regions_host(eng.model.ctx, eng.kv.c, S, h_cu, h_toks, None, 0.0, 1, h_acc, h_emit, h_nem,
                                       eng.ws.ptr, eng.ws.bytes, torch.cuda.current_stream().cuda_stream)
    B.check(rc, "hsd_verify_regions_host")
    assert mq == max_q
    for j, i in enumerate(sorted(orc)):
        a = int(per[i]["accept_len"])
        assert int(h_acc[j]) == a and int(h_nem[j]) == a + 1
        assert h_emit[j, :a + 1].tolist() == per[i]["emit"][:a + 1].tolist()
    after = eng.kv.seq_lens.cpu().numpy()
    assert (after - before).tolist() == [int(h_acc[j]) + 1 for j in range(S)]
    # malformed host offsets are refused before anything is launched
    bad = h_cu.clone(); bad[0] = 1
    rc, _ = B.hsd_verify_regions_host(eng.model.ctx, eng.kv.c, S, bad, h_toks, None, 0.0, 0, h_acc, h_emit, h_nem,
                                      eng.ws.ptr, eng.ws.bytes, torch.cuda.current_stream().cuda_stream)
    assert rc == B.HSD_ERR_INVALID_ARG


def test_layer_tap_returns_each_layers_residual_stream():
    """hsd_debug_tap: the residual stream after layer 0 of a 2-layer decoder equals the oracle's output for the same
    weights cut to one layer; after the last layer it is the buffer the LM head reads; a tap serves one forward."""
    import dataclasses
    import torch
    from oracle import hsd_oracle as O
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = I.small_decoder(2, 8192)
    wl = I.region_workload(seed=79, n_regions=2, prefix_lo=70, prefix_hi=140, draft_mean=30, draft_lo=8, draft_hi=60,
                           cfg=cfg)
    weights = I.make_weights(cfg, 9)
    dm = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(dm, [s.prefix_len + s.draft_len + 2 for s in wl.seqs], seed=2, poison=True)
    S = len(wl.seqs)
    T = sum(s.draft_len + 1 for s in wl.seqs)
    eng = R.Engine(dm, kv, max(sum(s.prefix_len for s in wl.seqs), T), S)
    first = eng.prefill([s.prefix_embeds for s in wl.seqs], [s.prefix_ids for s in wl.seqs]).cpu().numpy()
    drafts = [s.rand_tokens[:s.draft_len] for s in wl.seqs]
    toks, cu = I.pack_queries(first, drafts)
    taps = {}
    for layer in (0, 1):
        dst = torch.zeros(T, cfg.d_model, dtype=torch.float32, device=eng.dev)
        B.check(B.hsd_debug_tap(dm.ctx, layer, B.HSD_TAP_X, dst, dst.numel() * 4))
        eng.verify_regions(eng._i32(toks), eng._i32(cu), max(len(d) for d in drafts) + 1, T)
        eng.check_device("verify")
        taps[layer] = dst.cpu().numpy()
    st, ptr, nbytes = B.hsd_debug_buffer(dm.ctx, eng.ws.ptr, T, S, "x")
    assert st == 0 and nbytes == T * cfg.d_model * 4
    again = torch.zeros(T, cfg.d_model, dtype=torch.float32, device=eng.dev)       # not armed: stays zero
    eng.verify_regions(eng._i32(toks), eng._i32(cu), max(len(d) for d in drafts) + 1, T)
    torch.cuda.synchronize()
    assert float(again.abs().max()) == 0.0
    # a destination that is too small makes the forward refuse, and the tap is gone afterwards
    small = torch.zeros(16, dtype=torch.float32, device=eng.dev)
    B.check(B.hsd_debug_tap(dm.ctx, 1, B.HSD_TAP_X, small, 64))
    o = eng.alloc_outputs(S, max(len(d) for d in drafts) + 1, T)
    rc = B.hsd_verify_regions(dm.ctx, kv.c, S, eng._i32(cu), eng._i32(toks), None, max(len(d) for d in drafts) + 1, T, 0.0,
                              o["accept_len"], o["emit_tokens"], o["n_emit"], None, None, None, eng.ws.ptr, eng.ws.bytes,
                              torch.cuda.current_stream().cuda_stream)
    assert rc == B.HSD_ERR_WORKSPACE
    assert B.hsd_debug_tap(dm.ctx, 2, B.HSD_TAP_X, small, 64) == B.HSD_ERR_INVALID_ARG
    # oracle: the same first layer alone, and both layers
    for n_layers in (1, 2):
        cfg_n = dataclasses.replace(cfg, n_layers=n_layers)
        w_n = dict(weights, layers=weights["layers"][:n_layers])
        model = O.Decoder(cfg_n, w_n, np.float64)
        for i, s in enumerate(wl.seqs):
            cache = O.CachedSequence(model)
            cache.prefill(s.prefix_embeds, s.prefix_ids)
            x = model.embed_rows(None, np.concatenate([[first[i]], drafts[i]]))
            ref = cache.forward_rows(x, np.arange(len(x)), O.causal_allowed(len(x)))
            got = taps[n_layers - 1][cu[i]:cu[i + 1]]
            err = np.abs(got - ref).max() / np.abs(ref).max()
            assert err < 2e-2, (n_layers, i, err)


def test_wide_decoder_with_four_query_heads_per_kv_head_matches_oracle():
    """A wider decoder shape than the benchmark's (d_model 4096, 32 query / 8 kv heads x 64, FFN 8192: the width class of
    the 7-9 B parsers the paper evaluates, Sec. 4.3), one layer: 4096-wide RMSNorm rows, K = 4096 / 8192 projections,
    q-tiles of 32 tokens x 4 heads."""
    cfg = I.ModelConfig(n_layers=1, d_model=4096, n_heads=32, n_kv_heads=8, head_dim=64, d_ffn=8192, vocab=4096)
    wl = I.region_workload(seed=81, n_regions=3, prefix_lo=70, prefix_hi=200, draft_mean=40, draft_lo=8, draft_hi=100,
                           cfg=cfg, name="wide_regions")
    stats, orc, per, _ = run_region_parity(wl, 0)
    print("wide", stats, [(len(o.draft), o.res.accept_len) for o in orc.values()])
    assert stats["max_dz"] < H.LOGIT_TOL


def _decoder_hd128(n_layers=2, vocab=8192, qk_norm=False):
    """d_model 1024, 8 query / 4 kv heads x 128 (the head size of the 2-9 B decoders the paper evaluates, Sec. 4.3)."""
    return I.ModelConfig(n_layers=n_layers, d_model=1024, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=4096, vocab=vocab,
                         qk_norm=qk_norm)


@pytest.mark.parametrize("qk_norm", [False, True], ids=["plain", "qk_norm"])
def test_head_dim_128_regions_match_oracle(qk_norm):
    """Head dimension 128: two operand sub-tiles per Q / K / V tile, a 128-column accumulator, the rotation pairing
    dim i with dim i + 64 in the QKV epilogue, 256-byte KV rows.  Several q-tiles per sequence, ragged tails,
    prefixes that end inside a KV block, with and without the per-head RMSNorm of q and k."""
    wl = I.region_workload(seed=83, n_regions=5, prefix_lo=70, prefix_hi=330, draft_mean=60, draft_lo=8, draft_hi=200,
                           cfg=_decoder_hd128(qk_norm=qk_norm), name="hd128_regions")
    stats, orc, per, _ = run_region_parity(wl, 0)
    print("hd128", qk_norm, stats, [(len(o.draft), o.res.accept_len) for o in orc.values()])
    assert stats["max_dz"] < H.LOGIT_TOL


@pytest.mark.parametrize("plan", [(1 << 20, 1), (1, 1 << 20)], ids=["max_slices", "no_slices"])
def test_head_dim_128_kv_slicing_does_not_change_the_result(plan):
    wl = I.region_workload(seed=84, n_regions=4, prefix_lo=100, prefix_hi=520, draft_mean=50, draft_lo=8, draft_hi=150,
                           cfg=_decoder_hd128(), name="hd128_regions_slicing")
    stats, orc, per, _ = run_region_parity(wl, 0, attn_plan=plan)
    print("hd128 slicing", plan, stats)
    assert stats["max_dz"] < H.LOGIT_TOL


def test_head_dim_128_refuses_the_plain_cross_check_kernels():
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = _decoder_hd128(1, 4096)
    with pytest.raises(Exception):
        R.DeviceModel(cfg, I.make_weights(cfg, 1), B.HSD_FLAG_SIMT_ATTENTION)
