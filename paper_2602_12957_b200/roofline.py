"""Algorithmic work of one verify step and the roofline arithmetic used by the benchmark (host code only).

"Algorithmic" means what the method must move or compute: every streamed weight once, the K/V rows a query
can see once per layer, the new K/V rows written once, one embedding row per query token, and the tiny
outputs.  Activation round trips and padded tiles are not credited.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Sequence


@dataclass
class StepWork:
    total_q: int
    draft_tokens: int
    bytes: float
    flops: float
    gemm_flops: float
    attn_flops: float
    weight_bytes: float
    kv_read_bytes: float
    kv_write_bytes: float


def matmul_params(cfg) -> int:
    d, f = cfg.d_model, cfg.d_ffn
    per_layer = cfg.qkv_out * d + d * cfg.n_heads * cfg.head_dim + 2 * f * d + d * f
    return cfg.n_layers * per_layer + cfg.vocab * d


def step_work(cfg, context_lens: Sequence[int], q_lens: Sequence[int]) -> StepWork:
    """context_lens[i] = committed K/V rows of sequence i, q_lens[i] = its query rows (draft + 1)."""
    T = int(sum(q_lens))
    weight_bytes = 2.0 * cfg.streamed_params
    kvb = cfg.kv_bytes_per_token
    kv_read = kvb * float(sum(context_lens) + T)
    kv_write = kvb * float(T)
    embed = 2.0 * T * cfg.d_model
    outputs = 4.0 * (3 * T + 3 * len(q_lens))
    pairs = 0
    for L, q in zip(context_lens, q_lens):
        pairs += q * L + q * (q + 1) // 2          # row j sees L + j + 1 keys
    gemm = 2.0 * matmul_params(cfg) * T
    attn = 4.0 * cfg.n_heads * cfg.head_dim * cfg.n_layers * pairs
    return StepWork(T, T - len(q_lens), weight_bytes + kv_read + kv_write + embed + outputs, gemm + attn, gemm, attn,
                    weight_bytes, kv_read, kv_write)


def gemm_work(M: int, N: int, K: int, out_bytes_per_el: float = 2.0):
    """(flops, bytes) of C[M,N] = A[M,K] W[N,K]^T with bf16 operands."""
    return 2.0 * M * N * K, 2.0 * (M * K + N * K) + out_bytes_per_el * M * N


def roofline_time(nbytes: float, flops: float, bw_bytes_per_s: float, peak_flops_per_s: float) -> float:
    return max(nbytes / bw_bytes_per_s, flops / peak_flops_per_s)


def ridge(peak_flops_per_s: float, bw_bytes_per_s: float) -> float:
    return peak_flops_per_s / bw_bytes_per_s


def predicted_speedup(ai_base: float, flops_ratio: float, traffic_ratio: float, peak: float, bw: float) -> float:
    """Roofline-model speedup of a method that multiplies FLOPs by `flops_ratio` and memory traffic by
    `traffic_ratio` over a baseline of arithmetic intensity `ai_base` (time = max(bytes/bw, flops/peak))."""
    t_base = roofline_time(1.0, ai_base, bw, peak)
    t_new = roofline_time(traffic_ratio, ai_base * flops_ratio, bw, peak)
    return t_base / t_new
