"""The no-allocation LM-head entry point against the ordinary one.

Some callers of this library cannot call cudaMalloc where they run (inside another framework's stream-ordered
region, in a loop that must not touch the allocator, or after their whole memory budget has been handed out),
so `hsd_op_lm_head_argmax_noalloc` keeps its scratch in a fixed array inside the library.  The test calls it
twice in a row with different inputs — the shared array keeps the first call's contents, so the second call
only passes if the entry point clears what it reuses — and compares each result with the ordinary entry
point, which takes caller-provided scratch.  It also checks that a request beyond the fixed size is refused.

This file sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _inputs(cfg, rows, seed, device):
    import torch
    rng = np.random.default_rng(seed)
    h = I.bf16_round(rng.standard_normal((rows, cfg.d_model), dtype=np.float32))
    nxt = rng.integers(0, cfg.vocab, rows).astype(np.int32)
    return torch.from_numpy(h).to(device, torch.bfloat16), torch.from_numpy(nxt).to(device)


def _outputs(rows, device):
    import torch
    return (torch.full((rows,), -7, dtype=torch.int32, device=device),
            torch.full((rows,), -7.0, dtype=torch.float32, device=device),
            torch.full((rows,), -7.0, dtype=torch.float32, device=device))


def test_no_alloc_entry_point_matches_the_ordinary_one_twice_in_a_row():
    import torch
    from paper_2602_12957_b200 import binding as B
    from paper_2602_12957_b200 import runtime as R
    cfg = I.TINY
    model = R.DeviceModel(cfg, I.make_weights(cfg, 1), 0)
    dev = model.device
    stream = torch.cuda.current_stream().cuda_stream
    # the second call uses fewer rows and other data than the first: stale words of call 1 must not leak in; the third
    # fills the fixed array to its last word
    for rows, seed in ((300, 11), (77, 12), (B.HSD_NOALLOC_MAX_ROWS, 14)):
        h, nxt = _inputs(cfg, rows, seed, dev)
        am_ref, zm_ref, zd_ref = _outputs(rows, dev)
        scratch = torch.empty(rows, dtype=torch.int64, device=dev)
        B.check(B.hsd_op_lm_head_argmax(model.ctx, h, rows, nxt, scratch, rows * 8, am_ref, zm_ref, zd_ref, stream))
        am, zm, zd = _outputs(rows, dev)
        B.check(B.hsd_op_lm_head_argmax_noalloc(model.ctx, h, rows, nxt, am, zm, zd, stream))
        torch.cuda.synchronize()
        # same kernels, same tiles, same summation order: the two entry points agree to the bit
        assert np.array_equal(am.cpu().numpy(), am_ref.cpu().numpy())
        assert np.array_equal(zm.cpu().numpy(), zm_ref.cpu().numpy())
        assert np.array_equal(zd.cpu().numpy(), zd_ref.cpu().numpy())
        assert (am.cpu().numpy() >= 0).all() and (am.cpu().numpy() < cfg.vocab).all()
    # beyond the fixed array: a clear error, nothing launched, outputs untouched
    rows = B.HSD_NOALLOC_MAX_ROWS + 1
    h, nxt = _inputs(cfg, rows, 13, dev)
    am, zm, zd = _outputs(rows, dev)
    assert B.hsd_op_lm_head_argmax_noalloc(model.ctx, h, rows, nxt, am, zm, zd, stream) == B.HSD_ERR_TOO_LONG
    torch.cuda.synchronize()
    assert (am.cpu().numpy() == -7).all()
