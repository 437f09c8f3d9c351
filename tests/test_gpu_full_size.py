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
