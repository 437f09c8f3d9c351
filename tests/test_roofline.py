"""Host-side roofline arithmetic against the numbers the paper prints (supplement, FLOPs and Latency)."""
import os

from paper_2602_12957_b200 import inputs as I
from paper_2602_12957_b200 import roofline as RF

from .test_oracle_pins import read_golden


def test_a100_ridge_and_predicted_speedup_match_paper():
    g = read_golden()
    peak, bw = g["a100_peak_tflops"] * 1e12, g["a100_hbm_gbs"] * 1e9
    assert abs(RF.ridge(peak, bw) - g["a100_ridge"]) < 0.5
    s = RF.predicted_speedup(g["ai_baseline"], g["flops_ratio"], g["traffic_ratio"], peak, bw)
    assert abs(s - g["predicted_speedup"]) < 0.01
    # the method's own arithmetic intensity follows from the three ratios
    assert abs(g["ai_baseline"] * g["flops_ratio"] / g["traffic_ratio"] - g["ai_hsd"]) < 1.0
    # baseline decoding is memory-bound, the method is compute-bound on that machine
    assert g["ai_baseline"] < g["a100_ridge"] < g["ai_hsd"]


def test_step_work_constants_for_the_24_layer_decoder():
    c = I.DECODER
    assert RF.matmul_params(c) == 411_041_792
    w = RF.step_work(c, [1000], [1])
    assert abs(w.gemm_flops - 2 * 411_041_792) < 1
    assert w.attn_flops == 4 * 16 * 64 * 24 * 1001            # one row sees 1000 cached keys + itself
    assert w.kv_read_bytes == 49_152 * 1001 and w.kv_write_bytes == 49_152
    w2 = RF.step_work(c, [10, 20], [3, 2])
    assert w2.total_q == 5 and w2.draft_tokens == 3
    assert w2.attn_flops == 98_304 * ((11 + 12 + 13) + (21 + 22))
    f, b = RF.gemm_work(128, 256, 64)
    assert f == 2 * 128 * 256 * 64 and b == 2 * (128 * 64 + 256 * 64 + 128 * 256)
