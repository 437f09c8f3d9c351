"""GPU parity: whole verify step through the C-ABI against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

from . import harness as H

pytestmark = pytest.mark.gpu


def run_region_parity(wl, flags=0, dtype=np.float64, which=None):
    weights = I.make_weights(wl.cfg, wl.seed)
    orc = H.oracle_regions(wl, weights, dtype, which)
    per, eng, _ = H.gpu_regions(wl, weights, {i: o.pending for i, o in orc.items()},
                                {i: o.draft for i, o in orc.items()}, flags)
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


@pytest.mark.parametrize("flags", [2, 0], ids=["simt_attention", "tensor"])
def test_small_decoder_regions_match_oracle(flags):
    """Same layer shape as the 24-layer decoder (GQA 16/8, d 1024, FFN 4096), 2 layers, vocab 8192: several
    q-tiles per sequence, ragged tails, prefixes that end inside a KV block."""
    wl = I.region_workload(seed=77, n_regions=5, prefix_lo=70, prefix_hi=330, draft_mean=60, draft_lo=8, draft_hi=200,
                           cfg=I.small_decoder(2, 8192), name="small_regions")
    stats, orc, per, _ = run_region_parity(wl, flags)
    print("small", flags, stats, [(len(o.draft), o.res.accept_len) for o in orc.values()])
    assert stats["max_dz"] < H.LOGIT_TOL
