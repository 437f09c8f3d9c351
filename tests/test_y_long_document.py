"""Parity of the long-document configuration at full size: 24 layers, 2,048 visual rows + committed text up to 16,384
tokens, then one chunk of 1,024 and one of 2,048 draft tokens through hsd_verify_page, with the attention plan the
library chooses by itself (the KV range of every query tile is cut into slices whose partials are combined).

The float32 oracle needs a few minutes for this context (prefill of 16k rows through 24 layers, then two verify passes
over an 18k-token cache).  It therefore runs on a background thread that `conftest.py` starts when the GPU session
begins, while the other tests run; this file sorts late so that most of that work is done when the test asks for it.
Rows are teacher-forced, so the draft is random."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def test_long_document_full_size_chunks_over_a_long_context_match_oracle():
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = I.DECODER
    job = H.long_document_oracle()           # started at session start (or here, when this test runs alone)
    seq, draft, weights = job["seq"], job["draft"], job["weights"]
    L = seq.prefix_len
    dm = R.DeviceModel(cfg, weights, 0)
    kv = R.KvCache(dm, [L + 2049 + 64], seed=3, poison=True)
    eng = R.Engine(dm, kv, L, 1)
    eng.prefill([seq.prefix_embeds], [seq.prefix_ids])
    eng.check_device("prefill")
    outs = {}
    for k in (1024, 2048):                   # both chunks on the same committed state, default attention plan
        chunk = draft[:k]
        out = eng.verify_page(0, torch.tensor([job["pending"]()], dtype=torch.int32, device=eng.dev), eng._i32(chunk))
        eng.check_device("verify_page")
        g = {n: v.cpu().numpy() for n, v in out.items()}
        outs[k] = {"row_argmax": g["row_argmax"], "row_zmax": g["row_zmax"], "row_zdraft": g["row_zdraft"],
                   "accept_len": g["accept_len"][0], "n_emit": g["n_emit"][0], "emit": g["emit_tokens"][0]}
    res = job["results"]()                   # joins the oracle thread
    stats = {}
    for k in (1024, 2048):
        chunk, g = draft[:k], outs[k]
        H.compare_rows(f"long chunk {k}", res[k], chunk, g["row_argmax"][:k + 1], g["row_zmax"][:k + 1],
                       g["row_zdraft"][:k + 1], stats)
        H.compare_sequence(f"long chunk {k}", res[k], chunk, g["accept_len"], g["emit"], g["n_emit"],
                           g["row_argmax"][:k + 1], stats)
    print("full-size long", L, stats)
    assert L >= 16384 and stats["max_dz"] < H.LOGIT_TOL and stats["exact_rows"] > 1000
