"""Host-side checks of the seeded generators (no decoder arithmetic involved)."""
import numpy as np

from paper_2602_12957_b200 import inputs as I


def test_bf16_round_trip_and_nearest_even():
    a = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -0.3, 3.0e38, 0.0], np.float32)
    r = I.bf16_round(a)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0 + 2 ** -6)   # ties go to even mantissa
    assert np.array_equal(I.bf16_round(r), r)
    assert np.all(np.abs(r[:4] - a[:4]) <= np.abs(a[:4]) * 2.0 ** -8)
    assert np.array_equal(I.from_bf16_bits(I.to_bf16_bits(r)), r)


def test_weights_are_seeded_shaped_and_bf16_exact():
    w1, w2 = I.make_weights(I.TINY, 7), I.make_weights(I.TINY, 7)
    w3 = I.make_weights(I.TINY, 8)
    l = w1["layers"][0]
    assert l["w_qkv"].shape == (768, 256) and l["w_gate_up"].shape == (2048, 256) and l["w_down"].shape == (256, 1024)
    assert w1["lm_head"].shape == (4096, 256) and w1["embed"].shape == (4096, 256)
    assert np.array_equal(w1["lm_head"], w2["lm_head"]) and not np.array_equal(w1["lm_head"], w3["lm_head"])
    assert np.array_equal(I.bf16_round(l["w_o"]), l["w_o"])
    assert abs(float(l["w_qkv"].std()) - 0.02) < 1e-3 and abs(float(l["attn_norm"].mean()) - 1.0) < 0.01


def test_decoder_constants():
    c = I.DECODER
    assert c.streamed_params == 411_041_792 + 49 * 1024      # matrices + the 49 gain vectors
    assert c.kv_bytes_per_token == 49_152
    assert c.qkv_out == 2048


def test_workload_shapes():
    t = I.tiny_workload()
    assert len(t.seqs) == 4 and all(s.prefix_len == 128 and s.draft_len == 16 for s in t.seqs)
    assert all((s.prefix_ids[:64] == -1).all() and (s.prefix_ids[64:] >= 0).all() for s in t.seqs)
    assert all(0 <= s.agree_len <= 16 for s in t.seqs)
    r = I.region_workload(cfg=I.small_decoder())
    assert len(r.seqs) == 16
    assert all(256 <= s.prefix_len <= 1024 and 8 <= s.draft_len <= 256 and 0 <= s.agree_len <= s.draft_len for s in r.seqs)
    r2 = I.region_workload(cfg=I.small_decoder())
    assert [s.draft_len for s in r.seqs] == [s.draft_len for s in r2.seqs]
    m = I.mixed_workload(cfg=I.small_decoder(), fixed_draft_len=8)
    assert len(m.seqs) == 66 and sum(s.draft_len == 8 for s in m.seqs) == 64 and m.seqs[-1].draft_len == 1024


def test_lognormal_and_acceptance_statistics():
    rng = np.random.Generator(np.random.PCG64(1))
    k = I.lognormal_lengths(rng, 200_000, 64.0, 1, 10 ** 6)
    assert abs(k.mean() - 64.0) < 1.0
    rates = [I._agree_mixture(rng, 1000, 0.5, 0.2) / 1000 for _ in range(20000)]
    assert abs(np.mean(rates) - 0.8) < 0.01
    rates = [I._agree_mixture(rng, 1000, 0.75, 0.6) / 1000 for _ in range(20000)]
    assert abs(np.mean(rates) - 0.95) < 0.01
    rates = [I._agree_mixture(rng, 1000, 0.85, 0.6) / 1000 for _ in range(20000)]
    assert abs(np.mean(rates) - 0.97) < 0.01


def test_plant_draft():
    g = list(range(100, 110))
    rnd = np.array([1, 2, 103, 4, 5, 6], np.int32)
    d = I.plant_draft(g, 6, 3, rnd, 50000, False)
    assert list(d) == [100, 101, 102, 4, 5, 6]            # rnd[3] differs already; position 3 breaks agreement
    rnd2 = rnd.copy(); rnd2[3] = 103
    assert list(I.plant_draft(g, 6, 3, rnd2, 50000, False)) == [100, 101, 102, 104, 5, 6]   # equal -> bumped
    assert list(I.plant_draft(g, 6, 6, rnd, 50000, False)) == g[:6]
    assert list(I.plant_draft(g, 6, 2, rnd, 50000, True)) == [100, 101, 103, 103, 104, 105]
    assert list(I.plant_draft(g, 0, 0, rnd[:0], 50000, False)) == []


def test_block_tables_are_disjoint_and_padded():
    table, n = I.make_block_tables([130, 64, 1, 700], seed=3)
    used = table[table >= 0]
    assert len(used) == 3 + 1 + 1 + 11 and len(set(used.tolist())) == len(used) and used.max() < n
    assert (table[1, 1:] == -1).all()
    t2, _ = I.make_block_tables([130, 64, 1, 700], seed=3)
    assert np.array_equal(table, t2)


def test_pack_queries():
    toks, cu = I.pack_queries([7, 8], [np.array([1, 2, 3]), np.array([], np.int32)])
    assert list(toks) == [7, 1, 2, 3, 8] and list(cu) == [0, 4, 5]


def test_plant_tree_is_a_parent_first_prefix_tree_with_one_greedy_path():
    from collections import defaultdict
    from oracle import hsd_oracle as O
    greedy = list(range(500, 700))
    for seed in range(8):
        for n, a in ((1, 0), (1, 1), (5, 2), (40, 7), (127, 30)):
            tok, par, main = I.plant_tree(greedy, n, a, 1000, seed)
            assert tok.shape == (n,) and par.shape == (n + 1,) and par[0] == -1
            assert all(0 <= par[j] < j for j in range(1, n + 1))           # parents come first
            O.tree_depth_and_mask(par)                                     # the oracle accepts it
            kids = defaultdict(list)
            for j in range(1, n + 1):
                kids[int(par[j])].append(int(tok[j - 1]))
            assert all(len(set(v)) == len(v) for v in kids.values())       # siblings carry distinct tokens
            # the main path copies the greedy tokens for `a` steps and then leaves them
            a_eff = min(a, len(main))
            assert [int(tok[r - 1]) for r in main[:a_eff]] == greedy[:a_eff]
            assert all(par[main[d]] == (main[d - 1] if d else 0) for d in range(len(main)))
            if a_eff < len(main):
                assert int(tok[main[a_eff] - 1]) != greedy[a_eff]
            # walking the greedy tokens from the root follows the main path for exactly a_eff moves
            s, moves = 0, 0
            while True:
                nxt = [j for j in range(1, n + 1) if par[j] == s and int(tok[j - 1]) == greedy[moves]]
                if not nxt:
                    break
                s, moves = nxt[0], moves + 1
            assert moves == a_eff and (moves == 0 or s == main[moves - 1])
    t1, p1, _ = I.plant_tree(greedy, 40, 7, 1000, 3)
    t2, p2, _ = I.plant_tree(greedy, 40, 7, 1000, 3)
    assert np.array_equal(t1, t2) and np.array_equal(p1, p2)               # seeded
