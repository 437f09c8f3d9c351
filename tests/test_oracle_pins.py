"""Pins for the CPU oracle: each test fixes part of it against something other than itself —
a library decoder (whose rotary tables are float32, hence the 2e-7 bars), a library attention routine, closed forms, brute force, or numbers the paper prints."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import hsd_oracle as O
from paper_2602_12957_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_numbers.txt")
SMALL = I.ModelConfig(n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=128, vocab=97)


def read_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def small_model(seed=3, cfg=SMALL, dtype=np.float64):
    return O.Decoder(cfg, I.make_weights(cfg, seed), dtype)


def hf_llama(model):
    """The same decoder as a Hugging Face Llama (library routine)."""
    from transformers import LlamaConfig, LlamaForCausalLM
    c = model.cfg
    hc = LlamaConfig(vocab_size=c.vocab, hidden_size=c.d_model, intermediate_size=c.d_ffn,
                     num_hidden_layers=c.n_layers, num_attention_heads=c.n_heads,
                     num_key_value_heads=c.n_kv_heads, head_dim=c.head_dim, rms_norm_eps=c.rms_eps,
                     rope_theta=c.rope_base, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                     max_position_embeddings=4096, attn_implementation="eager")
    m = LlamaForCausalLM(hc).double().eval()
    W = model.weights
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    sd = {"model.embed_tokens.weight": t(W["embed"]), "model.norm.weight": t(W["final_norm"]),
          "lm_head.weight": t(W["lm_head"])}
    Hq, Hkv, D, f = c.n_heads, c.n_kv_heads, c.head_dim, c.d_ffn
    for i, lw in enumerate(W["layers"]):
        p = f"model.layers.{i}."
        sd[p + "input_layernorm.weight"] = t(lw["attn_norm"])
        sd[p + "post_attention_layernorm.weight"] = t(lw["ffn_norm"])
        sd[p + "self_attn.q_proj.weight"] = t(lw["w_qkv"][:Hq * D])
        sd[p + "self_attn.k_proj.weight"] = t(lw["w_qkv"][Hq * D:(Hq + Hkv) * D])
        sd[p + "self_attn.v_proj.weight"] = t(lw["w_qkv"][(Hq + Hkv) * D:])
        sd[p + "self_attn.o_proj.weight"] = t(lw["w_o"])
        sd[p + "mlp.gate_proj.weight"] = t(lw["w_gate_up"][:f])
        sd[p + "mlp.up_proj.weight"] = t(lw["w_gate_up"][f:])
        sd[p + "mlp.down_proj.weight"] = t(lw["w_down"])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


def mixed_prefix(model, n, n_visual, seed):
    rng = np.random.default_rng(seed)
    emb = np.zeros((n, model.cfg.d_model), np.float32)
    emb[:n_visual] = rng.standard_normal((n_visual, model.cfg.d_model)).astype(np.float32)
    ids = np.full(n, -1, np.int64)
    ids[n_visual:] = rng.integers(0, model.cfg.vocab, n - n_visual)
    return emb, ids


# ------------------------------------------------------------------ whole forward vs a library decoder
def oracle_full_logits(model, emb, ids):
    x = model.embed_rows(emb, ids)
    n = len(ids)
    return model.logits(O.decoder_forward(model, x, np.arange(n), O.causal_allowed(n)))


def library_input_rows(m, emb, ids):
    """Input rows built WITHOUT the oracle's `embed_rows`: token rows come from the library decoder's own embedding
    module fed with the id, visual rows (id < 0) are copied in by position."""
    ids = np.asarray(ids)
    x = torch.zeros(len(ids), m.config.hidden_size, dtype=torch.float64)
    with torch.no_grad():
        for r, t in enumerate(ids.tolist()):
            if t >= 0:
                x[r] = m.model.embed_tokens(torch.tensor(t))
            else:
                x[r] = torch.from_numpy(np.asarray(emb[r], np.float64))
    return x


def hf_logits(model, emb, ids):
    m = hf_llama(model)
    with torch.no_grad():
        if not np.any(np.asarray(ids) < 0):          # text only: the library gathers its own rows from the ids
            return m(input_ids=torch.from_numpy(np.asarray(ids, np.int64))[None]).logits[0].numpy()
        return m(inputs_embeds=library_input_rows(m, emb, ids)[None]).logits[0].numpy()


def test_forward_matches_library_llama():
    model = small_model()
    emb, ids = mixed_prefix(model, 23, 9, 1)
    z, zr = oracle_full_logits(model, emb, ids), hf_logits(model, emb, ids)
    assert z.shape == zr.shape == (23, SMALL.vocab)
    assert np.max(np.abs(z - zr)) < 2e-7


def test_forward_matches_library_llama_head_dim_64_mha():
    cfg = I.ModelConfig(n_layers=1, d_model=128, n_heads=2, n_kv_heads=2, head_dim=64, d_ffn=256, vocab=61)
    model = small_model(5, cfg)
    emb, ids = mixed_prefix(model, 17, 4, 2)
    assert np.max(np.abs(oracle_full_logits(model, emb, ids) - hf_logits(model, emb, ids))) < 2e-7


def interleaved_prefix(model, seed):
    """Visual and text rows interleaved, token id 0 and the largest id among the text rows, and an embedding row
    supplied (and to be ignored) at every text position."""
    rng = np.random.default_rng(seed)
    V = model.cfg.vocab
    ids = np.array([-1, -1, 0, 5, -1, V - 1, 0, 3, -1, -1, 11, 0], np.int64)
    emb = rng.standard_normal((len(ids), model.cfg.d_model)).astype(np.float32)
    return emb, ids


def test_input_rows_match_library_embedding_module():
    """`Decoder.embed_rows` against the library decoder's own embedding lookup: a text-only prefix goes in as
    input ids, a mixed one has its visual rows spliced in by the test; neither side of the comparison calls
    `embed_rows` except the oracle's."""
    model = small_model()
    m = hf_llama(model)
    emb, ids = interleaved_prefix(model, 21)
    x = model.embed_rows(emb, ids)
    assert np.array_equal(x, library_input_rows(m, emb, ids).numpy())
    assert np.array_equal(x[2], model.weights["embed"][0].astype(np.float64))          # id 0 is a token, not a visual row
    assert np.array_equal(x[0], emb[0].astype(np.float64)) and not np.array_equal(x[3], emb[3].astype(np.float64))
    z, zr = oracle_full_logits(model, emb, ids), hf_logits(model, emb, ids)
    assert np.max(np.abs(z - zr)) < 2e-7
    text = np.array([0, 7, 96, 0, 1, 50], np.int64)                                     # library fed with input_ids
    assert np.max(np.abs(oracle_full_logits(model, None, text) - hf_logits(model, None, text))) < 2e-7
    with pytest.raises(ValueError):
        model.embed_rows(None, np.array([3, -1]))


@pytest.mark.parametrize("mistake", ["rope_sign", "rope_pairing", "no_scale", "gqa_map", "mask_strict",
                                     "silu_on_up", "eps_outside", "no_residual_gain", "id_zero_is_visual",
                                     "embed_row_off_by_one", "visual_rows_from_table"])
def test_library_pin_catches_planted_mistakes(mistake, monkeypatch):
    """A plausible slip planted in the oracle (CPU only) must break the library pin."""
    model = small_model()
    emb, ids = interleaved_prefix(model, 3) if "id_zero" in mistake or "embed_row" in mistake or "visual_rows" in mistake \
        else mixed_prefix(model, 19, 6, 3)
    zr = hf_logits(model, emb, ids)
    if mistake == "rope_sign":
        def bad(x, pos, base):
            return O_rope(x, -pos, base)
        O_rope = O.rope
        monkeypatch.setattr(O, "rope", bad)
    elif mistake == "rope_pairing":          # interleaved (2i, 2i+1) pairing instead of rotate-half
        def bad(x, pos, base):
            D = x.shape[-1]
            inv = base ** (-np.arange(D // 2) * 2.0 / D)
            ang = pos[:, None] * inv[None]
            c, s = np.cos(ang)[:, None], np.sin(ang)[:, None]
            out = np.empty_like(x)
            out[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
            out[..., 1::2] = x[..., 1::2] * c + x[..., 0::2] * s
            return out
        monkeypatch.setattr(O, "rope", bad)
    elif mistake == "no_scale":
        monkeypatch.setattr(O.math, "sqrt", lambda v: 1.0)
    elif mistake == "gqa_map":               # head g reads kv head g % Hkv instead of g // group
        def bad(q, k, v, allowed):
            Hq, Hkv = q.shape[1], k.shape[1]
            idx = [g % Hkv for g in range(Hq)]
            return good(q, k[:, idx], v[:, idx], allowed)
        good = O.attention
        monkeypatch.setattr(O, "attention", bad)
    elif mistake == "mask_strict":
        def strict(n):                       # a row does not see itself (row 0 keeps itself to stay finite)
            m = np.tril(np.ones((n, n), bool), -1)
            m[0, 0] = True
            return m
        monkeypatch.setattr(O, "causal_allowed", strict)
    elif mistake == "silu_on_up":
        def bad(h, wgu, wd):
            f = wgu.shape[0] // 2
            gu = h @ wgu.T
            return (gu[:, :f] * O.silu(gu[:, f:])) @ wd.T
        monkeypatch.setattr(O, "swiglu_ffn", bad)
    elif mistake == "eps_outside":
        monkeypatch.setattr(O, "rmsnorm", lambda x, g, eps: x / (np.sqrt(np.mean(x * x, -1, keepdims=True)) + 1e-2) * g)
    elif mistake == "no_residual_gain":
        monkeypatch.setattr(O, "rmsnorm", lambda x, g, eps: x / np.sqrt(np.mean(x * x, -1, keepdims=True) + eps))
    elif mistake == "id_zero_is_visual":      # `ids <= 0` instead of `ids < 0` selects the visual row
        def bad(self, embeds, ids_):
            ids_ = np.asarray(ids_)
            x = self.w(self.weights["embed"][np.maximum(ids_, 0)])
            return np.ascontiguousarray(np.where((ids_ <= 0)[:, None], self.w(np.asarray(embeds)), x))
        monkeypatch.setattr(O.Decoder, "embed_rows", bad)
    elif mistake == "embed_row_off_by_one":   # table row id + 1
        def bad(self, embeds, ids_):
            ids_ = np.asarray(ids_)
            x = self.w(self.weights["embed"][np.minimum(np.maximum(ids_, 0) + 1, self.cfg.vocab - 1)])
            return np.ascontiguousarray(np.where((ids_ < 0)[:, None], self.w(np.asarray(embeds)), x))
        monkeypatch.setattr(O.Decoder, "embed_rows", bad)
    elif mistake == "visual_rows_from_table": # the given rows are ignored
        def bad(self, embeds, ids_):
            return np.ascontiguousarray(self.w(self.weights["embed"][np.maximum(np.asarray(ids_), 0)]))
        monkeypatch.setattr(O.Decoder, "embed_rows", bad)
    z = oracle_full_logits(model, emb, ids)
    assert np.max(np.abs(z - zr)) > 1e-4


# ------------------------------------------------------------------ attention vs library + closed form
def test_attention_matches_torch_sdpa_gqa_arbitrary_mask():
    rng = np.random.default_rng(0)
    Tq, Tk, Hq, Hkv, D = 7, 13, 6, 2, 16
    q, k, v = rng.standard_normal((Tq, Hq, D)), rng.standard_normal((Tk, Hkv, D)), rng.standard_normal((Tk, Hkv, D))
    allowed = rng.random((Tq, Tk)) < 0.6
    allowed[:, 0] = True
    got = O.attention(q, k, v, allowed)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(allowed)[None, None],
                                                           enable_gqa=True)[0].permute(1, 0, 2).numpy()
    assert np.max(np.abs(got - ref)) < 1e-12


def test_attention_uniform_keys_gives_mean_of_values():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((3, 2, 8))
    k = np.tile(rng.standard_normal((1, 1, 8)), (5, 1, 1))
    v = rng.standard_normal((5, 1, 8))
    out = O.attention(q, k, v, np.ones((3, 5), bool))
    assert np.allclose(out, np.broadcast_to(v.mean(0)[None], (3, 2, 8)), atol=1e-13)


def test_attention_single_allowed_key_copies_its_value():
    rng = np.random.default_rng(2)
    q, k, v = rng.standard_normal((4, 2, 8)), rng.standard_normal((6, 2, 8)), rng.standard_normal((6, 2, 8))
    allowed = np.zeros((4, 6), bool)
    allowed[np.arange(4), [5, 0, 3, 2]] = True
    out = O.attention(q, k, v, allowed)
    assert np.allclose(out, v[[5, 0, 3, 2]], atol=1e-13)


# ------------------------------------------------------------------ RoPE / RMSNorm / SiLU closed forms
def test_rope_closed_forms():
    rng = np.random.default_rng(4)
    D = 64
    x = rng.standard_normal((5, 3, D))
    assert np.array_equal(O.rope(x, np.zeros(5), 10000.0), x)                     # position 0 = identity
    y = O.rope(x, np.array([0, 1, 7, 100, 4000]), 10000.0)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))     # rotation keeps norms
    # pair (0, D/2) has frequency base^0 = 1: a plain rotation by `pos` radians
    p = 7.0
    e = np.zeros((1, 1, D)); e[0, 0, 0] = 1.0
    r = O.rope(e, np.array([p]), 10000.0)[0, 0]
    assert abs(r[0] - math.cos(p)) < 1e-15 and abs(r[D // 2] - math.sin(p)) < 1e-15
    assert np.count_nonzero(np.abs(r) > 1e-15) == 2
    # pair (i, i + D/2) has frequency base^(-2i/D)
    i = 5
    e = np.zeros((1, 1, D)); e[0, 0, i + D // 2] = 1.0
    r = O.rope(e, np.array([p]), 10000.0)[0, 0]
    th = p * 10000.0 ** (-2 * i / D)
    assert abs(r[i] + math.sin(th)) < 1e-15 and abs(r[i + D // 2] - math.cos(th)) < 1e-15
    # relative-position property
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    dots = [float(np.sum(O.rope(q, np.array([m]), 1e4) * O.rope(k, np.array([m - 11]), 1e4))) for m in (11, 50, 999)]
    assert max(dots) - min(dots) < 1e-9


def test_rmsnorm_closed_forms_and_library():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((6, 32)) * 3.0
    g = 1.0 + 0.1 * rng.standard_normal(32)
    y = O.rmsnorm(x, np.ones(32), 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, -1)), 1.0)
    assert np.allclose(O.rmsnorm(17.0 * x, g, 0.0), O.rmsnorm(x, g, 0.0))
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), 1e-6).numpy()
    assert np.max(np.abs(O.rmsnorm(x, g, 1e-6) - ref)) < 1e-13
    assert np.allclose(O.rmsnorm(np.full((1, 4), 2.0), np.arange(1.0, 5.0), 0.0), np.arange(1.0, 5.0))


def test_silu_and_swiglu():
    x = np.linspace(-6, 6, 41)
    assert np.max(np.abs(O.silu(x) - torch.nn.functional.silu(torch.from_numpy(x)).numpy())) < 1e-14
    assert O.silu(np.array([0.0]))[0] == 0.0
    # one hidden unit, hand-computed: gate 2, up 3, down 5 on input 1 -> silu(2) * 3 * 5
    out = O.swiglu_ffn(np.array([[1.0]]), np.array([[2.0], [3.0]]), np.array([[5.0]]))
    assert abs(out[0, 0] - (2.0 / (1.0 + math.exp(-2.0))) * 15.0) < 1e-14


def test_logits_closed_form_when_branches_are_zero():
    """With W_o = 0 and W_down = 0 every layer is the identity, so logits = RMSNorm(input row) W_lm^T."""
    model = small_model()
    for lw in model.weights["layers"]:
        lw["w_o"] = np.zeros_like(lw["w_o"])
        lw["w_down"] = np.zeros_like(lw["w_down"])
    emb, ids = mixed_prefix(model, 9, 3, 6)
    z = oracle_full_logits(model, emb, ids)
    x = model.embed_rows(emb, ids)
    g = model.weights["final_norm"].astype(np.float64)
    ref = (x / np.sqrt((x * x).mean(-1, keepdims=True) + SMALL.rms_eps) * g) @ model.weights["lm_head"].astype(np.float64).T
    assert np.max(np.abs(z - ref)) < 1e-12


# ------------------------------------------------------------------ the verification step itself
def prefilled(model, emb, ids):
    seq = O.CachedSequence(model)
    pending = seq.prefill(emb, ids, chunk=5)       # ragged chunks on purpose
    return seq, pending


def test_prefill_first_token_is_library_argmax():
    model = small_model()
    emb, ids = mixed_prefix(model, 21, 8, 7)
    _, pending = prefilled(model, emb, ids)
    assert pending == int(np.argmax(hf_logits(model, emb, ids)[-1]))


def test_verify_rows_equal_library_teacher_forced_logits():
    """Row j of a verify call is the decoder's distribution after [prefix, pending, d_1..d_j] (Eq. 8)."""
    model = small_model()
    emb, ids = mixed_prefix(model, 15, 5, 8)
    seq, pending = prefilled(model, emb, ids)
    draft = np.random.default_rng(0).integers(0, SMALL.vocab, 6)
    res_c = O.verify_cached(seq, pending, draft, keep_logits=True)
    res_f = O.verify_full(model, emb, ids, pending, draft, keep_logits=True)
    all_ids = np.concatenate([ids, [pending], draft])
    all_emb = np.concatenate([emb, np.zeros((7, SMALL.d_model), np.float32)])
    zr = hf_logits(model, all_emb, all_ids)[len(ids):]
    assert np.max(np.abs(res_f.logits - zr)) < 2e-7
    assert np.max(np.abs(res_c.logits - zr)) < 2e-7
    assert np.array_equal(res_c.row_argmax, zr.argmax(1))
    assert np.allclose(res_c.row_zdraft[:6], zr[np.arange(6), draft])
    assert np.isnan(res_c.row_zdraft[6])
    srt = np.sort(zr, axis=1)
    assert np.allclose(res_c.row_gap, srt[:, -1] - srt[:, -2]) and np.allclose(res_c.row_zmax, srt[:, -1])


def test_own_greedy_continuation_is_fully_accepted_with_bonus():
    model = small_model()
    emb, ids = mixed_prefix(model, 12, 4, 9)
    seq, pending = prefilled(model, emb, ids)
    k = 7
    g = O.greedy_continuation(seq, pending, k + 1)
    assert seq.length == 12                                            # cache untouched
    for verify in (lambda d: O.verify_cached(seq, pending, d), lambda d: O.verify_full(model, emb, ids, pending, d)):
        res = verify(np.array(g[:k]))
        assert res.accept_len == k and len(res.emitted) == k + 1
        assert res.emitted == g[:k + 1]                                # k draft tokens + the bonus token


def test_greedy_continuation_is_library_greedy_decode():
    model = small_model()
    emb, ids = mixed_prefix(model, 10, 3, 10)
    seq, pending = prefilled(model, emb, ids)
    g = O.greedy_continuation(seq, pending, 4)
    cur_ids, cur_emb = ids.copy(), emb.copy()
    tok = pending
    for j in range(4):
        cur_ids = np.concatenate([cur_ids, [tok]])
        cur_emb = np.concatenate([cur_emb, np.zeros((1, SMALL.d_model), np.float32)])
        tok = int(np.argmax(hf_logits(model, cur_emb, cur_ids)[-1]))
        assert tok == g[j]


def test_wrong_first_token_accepts_nothing_and_emits_models_token():
    model = small_model()
    emb, ids = mixed_prefix(model, 12, 4, 11)
    seq, pending = prefilled(model, emb, ids)
    g = O.greedy_continuation(seq, pending, 5)
    draft = np.array(g)
    draft[0] = (draft[0] + 1) % SMALL.vocab
    res = O.verify_cached(seq, pending, draft)
    assert res.accept_len == 0 and res.emitted == [g[0]]


@pytest.mark.parametrize("a", [0, 1, 3, 6])
def test_planted_agreement_length_is_recovered(a):
    model = small_model()
    emb, ids = mixed_prefix(model, 12, 4, 12)
    seq, pending = prefilled(model, emb, ids)
    k = 6
    g = O.greedy_continuation(seq, pending, k + 1)
    rnd = np.random.default_rng(a).integers(0, SMALL.vocab, k).astype(np.int32)
    d = I.plant_draft(g, k, a, rnd, SMALL.vocab, continue_on_greedy=False)
    res = O.verify_cached(seq, pending, d)
    assert res.accept_len == a
    assert res.emitted == g[:a + 1]


def test_empty_draft_is_one_plain_decode_step():
    model = small_model()
    emb, ids = mixed_prefix(model, 9, 2, 13)
    seq, pending = prefilled(model, emb, ids)
    res = O.verify_cached(seq, pending, np.zeros(0, np.int64))
    assert res.accept_len == 0 and len(res.emitted) == 1
    assert res.emitted[0] == O.greedy_continuation(seq, pending, 1)[0]


def test_teacher_forcing_later_tokens_do_not_change_earlier_rows():
    model = small_model()
    emb, ids = mixed_prefix(model, 9, 2, 14)
    seq, pending = prefilled(model, emb, ids)
    d1 = np.array([3, 9, 27, 81, 5])
    d2 = d1.copy(); d2[3] = 44
    z1 = O.verify_cached(seq, pending, d1, keep_logits=True).logits
    z2 = O.verify_cached(seq, pending, d2, keep_logits=True).logits
    assert np.array_equal(z1[:4], z2[:4])          # rows 0..3 see tokens d_1..d_3 only
    assert not np.allclose(z1[4], z2[4])


def test_commit_rollback_then_next_step_equals_stateless():
    """verify -> commit (pending + accepted rows) -> verify again == stateless forward on the accepted text."""
    model = small_model()
    emb, ids = mixed_prefix(model, 11, 4, 15)
    seq, pending = prefilled(model, emb, ids)
    g = O.greedy_continuation(seq, pending, 9)
    d = I.plant_draft(g, 5, 2, np.array([1, 2, 3, 4, 5], np.int32), SMALL.vocab, False)
    res = O.verify_cached(seq, pending, d)
    assert res.accept_len == 2
    new_pending = O.commit_step(seq, res)
    assert seq.length == 11 + 1 + 2 and new_pending == g[2]
    d2 = np.array(g[3:7])
    r_c = O.verify_cached(seq, new_pending, d2, keep_logits=True)
    ids2 = np.concatenate([ids, [pending], g[:2]])
    emb2 = np.concatenate([emb, np.zeros((3, SMALL.d_model), np.float32)])
    r_f = O.verify_full(model, emb2, ids2, new_pending, d2, keep_logits=True)
    assert np.max(np.abs(r_c.logits - r_f.logits)) < 2e-7
    assert r_c.accept_len == 4 and r_c.emitted == g[3:8]


def test_chunk_size_invariance():
    """A page draft verified in chunks of 3 or of 7 gives the same text."""
    model = small_model()
    emb, ids = mixed_prefix(model, 10, 4, 16)
    n = 21

    def run(chunk, subs):
        seq, pending = prefilled(model, emb, ids)
        g = [pending] + O.greedy_continuation(seq, pending, n + 2)
        draft = np.array(g[1:n + 1])
        for s in subs:
            draft[s] = (draft[s] + 1) % SMALL.vocab
        out, cur, steps = [], 0, 0
        while cur < n:
            d = draft[cur:cur + chunk]
            res = O.verify_cached(seq, pending, d)
            pending = O.commit_step(seq, res)
            out.extend(res.emitted)
            cur += res.accept_len + 1       # a substitution error: the draft re-aligns after the correction
            steps += 1
        return out[:n], steps

    a, steps_a = run(3, [4, 13])
    b, steps_b = run(7, [4, 13])
    seq, pending = prefilled(model, emb, ids)
    g = O.greedy_continuation(seq, pending, n)
    assert a == g and b == g and steps_b < steps_a


# ------------------------------------------------------------------ tree form (Eq. 5-9) against chains
def test_chain_is_the_one_candidate_tree():
    depth, allowed = O.tree_depth_and_mask(O.chain_parents(5))
    assert np.array_equal(depth, np.arange(6))
    assert np.array_equal(allowed, np.tril(np.ones((6, 6), bool)))


def test_tree_rows_equal_each_candidate_verified_alone():
    """Packed tree + ancestry mask gives, at every node v, the logits of the chain pi(v) (Eq. 8)."""
    model = small_model()
    emb, ids = mixed_prefix(model, 8, 3, 17)
    seq, pending = prefilled(model, emb, ids)
    #        root -> 5 -> 6 -> 7
    #                  \-> 9
    #             -> 11 -> 12
    tokens = np.array([5, 6, 7, 9, 11, 12])
    parent = np.array([-1, 0, 1, 2, 1, 0, 5])
    zt = O.verify_cached(seq, pending, tokens, parent, keep_logits=True).logits
    paths = {3: [5, 6, 7], 4: [5, 9], 6: [11, 12]}
    rows = {3: [1, 2, 3], 4: [1, 4], 6: [5, 6]}
    for leaf, toks in paths.items():
        zc = O.verify_cached(seq, pending, np.array(toks), keep_logits=True).logits
        assert np.max(np.abs(zc[0] - zt[0])) < 2e-7
        for j, r in enumerate(rows[leaf]):
            assert np.max(np.abs(zc[j + 1] - zt[r])) < 2e-7


def literal_traverse(dist, C, log_tau):
    """Literal walk over prefixes: Next(v) from Eq. 7 on the candidate set C, u* Eq. 9, u_hat Eq. 10,
    test Eq. 11, result Eq. 12.  `dist(prefix_tuple)` returns the logits after that prefix."""
    pi = ()
    while True:
        z = dist(pi)
        u_hat = min(range(len(z)), key=lambda u: (-z[u], u))
        nxt = sorted({c[len(pi)] for c in C if len(c) > len(pi) and tuple(c[:len(pi)]) == pi})
        if not nxt:
            return list(pi) + [u_hat]
        u_star = min(nxt, key=lambda u: (-z[u], u))
        ok = (u_star == u_hat) if log_tau == 0.0 else (z[u_star] - z[u_hat] >= log_tau)
        if not ok:
            return list(pi) + [u_hat]
        pi = pi + (u_star,)


def build_tree(C):
    """Prefix tree of candidate set C as (tokens, parent) with row 0 the root."""
    nodes = {(): 0}
    tokens, parent = [], [-1]
    for c in sorted(set(map(tuple, C))):
        for i in range(1, len(c) + 1):
            p = c[:i]
            if p not in nodes:
                nodes[p] = len(parent)
                parent.append(nodes[p[:-1]])
                tokens.append(p[-1])
    return np.array(tokens, np.int64), np.array(parent, np.int64)


@pytest.mark.parametrize("log_tau", [0.0, math.log(0.75), math.log(0.3)])
def test_brute_force_all_drafts_tiny_vocab(log_tau):
    """Enumerate every draft of length 0..3 over a 5-token vocabulary (and pairs of them as 2-candidate trees)
    and compare with the literal prefix walk on a table of fixed logits per prefix."""
    V = 5
    rng = np.random.default_rng(21)
    table = {}

    def dist(prefix):
        if prefix not in table:
            z = rng.standard_normal(V)
            if len(prefix) == 1:
                z[2] = z[3] = z.max() + 0.01        # an exact tie for the top score
            table[prefix] = z
        return table[prefix]

    drafts = [d for k in range(4) for d in itertools.product(range(V), repeat=k)]
    cand_sets = [[d] for d in drafts] + [[a, b] for a in drafts[1::7] for b in drafts[2::5]]
    checked = 0
    for C in cand_sets:
        tokens, parent = build_tree(C)
        prefixes = [()]
        for j in range(1, len(parent)):
            prefixes.append(prefixes[parent[j]] + (int(tokens[j - 1]),))
        logits = np.stack([dist(p) for p in prefixes])
        path, emitted = O.greedy_traverse(logits, np.concatenate([[-1], tokens]), parent, log_tau)
        assert emitted == literal_traverse(dist, [c for c in C], log_tau)
        assert len(emitted) == len(path) + 1
        checked += 1
    assert checked > 300


def test_threshold_rule_closed_form():
    """Eq. 11 on probabilities == the same test on raw logits (the softmax normaliser cancels), and tau -> 1
    with a unique maximum == exact match."""
    rng = np.random.default_rng(22)
    for _ in range(200):
        z = rng.standard_normal(11) * 2
        p = np.exp(z - z.max()); p /= p.sum()
        u, tau = int(rng.integers(0, 11)), float(rng.uniform(0.05, 0.999))
        lhs = math.log(p[u]) - math.log(p.max()) >= math.log(tau)
        _, em = O.greedy_traverse(z[None].repeat(2, 0), np.array([-1, u]), np.array([-1, 0]), math.log(tau))
        assert (len(em) == 2) == lhs
        _, em1 = O.greedy_traverse(z[None].repeat(2, 0), np.array([-1, u]), np.array([-1, 0]), 0.0)
        assert (len(em1) == 2) == (u == int(np.argmax(z)))


def test_step_count_identity_matches_papers_printed_numbers():
    """Each step emits accepted + 1 tokens (Eq. 12), so forward passes per token = 1 / (AAL + 1).
    The paper prints AAL 4.55 (Table 1) and a forward-pass ratio of 0.179 (supplement); they agree."""
    g = read_golden()
    assert abs(1.0 / (g["aal_hunyuanocr"] + 1.0) - g["forward_pass_ratio"]) < 0.002
    # and the oracle's own stepping obeys the identity exactly
    model = small_model()
    emb, ids = mixed_prefix(model, 8, 3, 18)
    seq, pending = prefilled(model, emb, ids)
    n = 30
    gcont = O.greedy_continuation(seq, pending, n + 8)
    draft = np.array(gcont[:n]);
    for s in (3, 4, 11, 20):
        draft[s] = (draft[s] + 1) % SMALL.vocab
    cur, steps, acc, emitted = 0, 0, 0, 0
    while cur < n:
        res = O.verify_cached(seq, pending, draft[cur:cur + 6])
        pending = O.commit_step(seq, res)
        steps += 1; acc += res.accept_len; emitted += len(res.emitted)
        cur += res.accept_len + 1
    assert emitted == acc + steps
    assert abs(steps / emitted - 1.0 / (acc / steps + 1.0)) < 1e-12


def test_float32_mode_tracks_float64():
    m64, m32 = small_model(), small_model(dtype=np.float32)
    emb, ids = mixed_prefix(m64, 12, 4, 19)
    z64, z32 = oracle_full_logits(m64, emb, ids), oracle_full_logits(m32, emb, ids)
    assert z32.dtype == np.float32 and np.max(np.abs(z64 - z32)) < 1e-4


# ------------------------------------------------------------------ per-head QK-norm vs a library decoder that has it
def hf_qwen3(model):
    """The decoder with per-head q/k RMSNorm as a Hugging Face Qwen3 (library routine)."""
    from transformers import Qwen3Config, Qwen3ForCausalLM
    c = model.cfg
    hc = Qwen3Config(vocab_size=c.vocab, hidden_size=c.d_model, intermediate_size=c.d_ffn,
                     num_hidden_layers=c.n_layers, num_attention_heads=c.n_heads,
                     num_key_value_heads=c.n_kv_heads, head_dim=c.head_dim, rms_norm_eps=c.rms_eps,
                     rope_theta=c.rope_base, attention_bias=False, tie_word_embeddings=False,
                     max_position_embeddings=4096, use_sliding_window=False, attn_implementation="eager")
    m = Qwen3ForCausalLM(hc).double().eval()
    W = model.weights
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    sd = {"model.embed_tokens.weight": t(W["embed"]), "model.norm.weight": t(W["final_norm"]),
          "lm_head.weight": t(W["lm_head"])}
    Hq, Hkv, D, f = c.n_heads, c.n_kv_heads, c.head_dim, c.d_ffn
    for i, lw in enumerate(W["layers"]):
        p = f"model.layers.{i}."
        sd[p + "input_layernorm.weight"] = t(lw["attn_norm"])
        sd[p + "post_attention_layernorm.weight"] = t(lw["ffn_norm"])
        sd[p + "self_attn.q_proj.weight"] = t(lw["w_qkv"][:Hq * D])
        sd[p + "self_attn.k_proj.weight"] = t(lw["w_qkv"][Hq * D:(Hq + Hkv) * D])
        sd[p + "self_attn.v_proj.weight"] = t(lw["w_qkv"][(Hq + Hkv) * D:])
        sd[p + "self_attn.o_proj.weight"] = t(lw["w_o"])
        sd[p + "self_attn.q_norm.weight"] = t(lw["q_norm"])
        sd[p + "self_attn.k_norm.weight"] = t(lw["k_norm"])
        sd[p + "mlp.gate_proj.weight"] = t(lw["w_gate_up"][:f])
        sd[p + "mlp.up_proj.weight"] = t(lw["w_gate_up"][f:])
        sd[p + "mlp.down_proj.weight"] = t(lw["w_down"])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


def test_qk_norm_forward_matches_library_qwen3_and_changes_the_result():
    cfg = I.ModelConfig(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=256, vocab=61, qk_norm=True)
    model = small_model(7, cfg)
    emb, ids = mixed_prefix(model, 19, 5, 3)
    z = oracle_full_logits(model, emb, ids)
    m = hf_qwen3(model)
    x = torch.from_numpy(model.embed_rows(emb, ids))[None]
    with torch.no_grad():
        zr = m(inputs_embeds=x).logits[0].numpy()
    assert np.max(np.abs(z - zr)) < 2e-7
    # the cached form agrees with the stateless one, and without the norm the logits differ
    cache = O.CachedSequence(model)
    cache.prefill(emb, ids)
    assert np.max(np.abs(cache.last_prefill_logits - z[-1])) < 1e-9
    plain = I.ModelConfig(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=256, vocab=61)
    model_p = O.Decoder(plain, model.weights, np.float64)
    assert np.max(np.abs(oracle_full_logits(model_p, emb, ids) - z)) > 1e-3
