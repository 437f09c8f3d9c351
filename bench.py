#!/usr/bin/env python
"""Benchmark of the HSD draft-verification step on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (one process per GPU)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands, on host cores

One step = one pass of the whole hot path over one batch: pack/embed, 24 x (norm, QKV+RoPE+KV write, paged
causal attention, O, norm, gate/up+SwiGLU, down), final norm, LM head + argmax + draft logit, accept/emit,
KV commit.  The line's own numbers are the region-level stage: 16 regions per GPU, prefixes 256-1024 visual rows,
lognormal draft lengths (mean 64, clipped 8-256), planted agreement with mean acceptance 0.8, paged KV with
64-token blocks and shuffled physical blocks.  At one GPU the same run also times one step of every other
configuration (short drafts, page chunk, long-document chunks, mixed batch, candidate trees) under `workloads`.
Inputs are synthetic and seeded; weights are random-init.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_12957_b200 import inputs as I          # noqa: E402
from paper_2602_12957_b200 import roofline as RF       # noqa: E402
from paper_2602_12957_b200 import shard as SH          # noqa: E402

METRIC = "draft tokens verified per second (verify step: forward over paged prefix + accept + KV commit)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel classes, from the ncu
# captures summarised under profiles/, per workload; a class is absent (-> null) when its kernel has changed since
# its counters were taken, or when no capture of that workload exists.
NCU_TRAFFIC_BYTES = {
    "region": {"attention": 30_975_744 + 4_352, "gemm_gate_up": 19_522_048, "gemm_qkv": 7_284_992 + 1_280,
               "gemm_o": 10_249_984, "gemm_down": 24_669_696},
    "long2048": {"attention": 42_460_928 + 4_530_176},
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"])}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,utilization.gpu,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        rows = []
        for line in open(self.tmp.name):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                rows.append((float(parts[0]), float(parts[1]), float(parts[2]), float(parts[3]), parts[4:8]))
            except ValueError:
                continue
        os.unlink(self.tmp.name)
        load = [r for r in rows if r[3] >= 50.0] or rows
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in load:
            for n, v in zip(names, r[4]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median([r[0] for r in load])) if load else None,
                "sm_max_mhz": load[0][1] if load else None,
                "power_w_max": max([r[2] for r in load]) if load else None,
                "reasons": sorted(reasons), "samples": len(load)}


# ------------------------------------------------------------------------------------------------ workloads
WORKLOADS = {
    "region": "region-level stage: 24-layer decoder d1024 16q/8kv x64 ffn4096 vocab32768, 16 regions per GPU, prefix "
              "256-1024, lognormal drafts mean 64 (8-256), acceptance 0.8, paged KV block 64",
    "region_short": "region-level stage, short drafts (the memory-bound regime): the same 16 regions, every draft 8 tokens "
                    "(144 query rows)",
    "page": "page-level stage, last chunk of the schedule: batch 1, 7936 committed tokens (4096 visual + 256 prompt + "
            "3584 accepted), chunk of 512 draft tokens",
    "long1024": "long-document page verify, last chunk of the schedule: batch 1, 17408 committed tokens, chunk of 1024",
    "long2048": "long-document page verify, last chunk of the schedule: batch 1, 16384 committed tokens, chunk of 2048",
    "tree": "one step of the decoupled-verification loop on the region batch's 16 prefixes (256-1024): window matching "
            "(n = 3) against two damaged copies of each region's text and prefix-tree packing on the device (128 rows "
            "per sequence), tree verification at tau 0.75, compaction of the accepted path's K/V rows",
    "region_hd128": "region-level stage on a wider decoder with 128-wide heads (the head size of the 2-9 B parsers of "
                    "Sec. 4.3): 8 layers, d2048 16q/8kv x128 ffn8192 vocab32768, the same 16 regions and drafts",
    "mixed": "mixed serving batch: 64 regions (prefix 128-2048, lognormal drafts mean 96, 8-512) + 2 page chunks of 1024 "
             "over 4352-token prefixes, one varlen launch",
}
EXTRA_WORKLOADS = ["region_short", "page", "long1024", "long2048", "mixed", "tree", "region_hd128"]
# the second decoder shape (a slice of 8 layers keeps the host-side weight draw short; per-layer work is what is measured)
DECODER_HD128 = I.ModelConfig(n_layers=8, d_model=2048, n_heads=16, n_kv_heads=8, head_dim=128, d_ffn=8192, vocab=32768)


def workload_cfg(name):
    return DECODER_HD128 if name == "region_hd128" else I.DECODER

TREE_NODES = 127     # nodes below the root: 128 packed rows per sequence, the paper's packing limit (Sec. 4.3)
TREE_MAIN = 64       # the planted agreement lengths of the region workload are scaled to this many tokens
WINDOW_N = 3         # reference window (Sec. 4.3)
LOG_TAU_TREE = float(np.log(0.75))
PAGE_SHAPES = {"page": (7936, 512), "long1024": (17408, 1024), "long2048": (16384, 2048)}


def make_workload(name, rank, world=1, sharded=False, mixed_k=0):
    """The seeded workload of this rank.  Returns (workload, plant): `plant` says whether the drafts are planted along
    the library's own greedy path (region) or random (the others: kernel time does not depend on token values)."""
    cfg = workload_cfg(name)
    if name in ("region", "region_short", "tree", "region_hd128"):
        fixed = 8 if name == "region_short" else None
        if sharded and world > 1:       # ONE batch of 16 x world regions, split by the cost model
            wl = I.region_workload(seed=I.BASE_SEED + 1, n_regions=16 * world, fixed_draft_len=fixed, cfg=cfg)
            own = SH.partition([s.prefix_len for s in wl.seqs], [s.draft_len for s in wl.seqs], world)[rank]
            wl.seqs = [wl.seqs[i] for i in own]
        else:
            wl = I.region_workload(seed=I.BASE_SEED + 1 + 1000 * rank, fixed_draft_len=fixed, cfg=cfg)
        if name == "tree":
            for s_ in wl.seqs:      # same prefixes; the draft becomes a 127-node tree whose main path agrees as planted
                s_.agree_len = int(round(TREE_MAIN * s_.agree_len / max(1, s_.draft_len)))
                s_.draft_len = TREE_NODES
        wl.name = name
        return wl, name in ("region", "tree")
    if name == "mixed":
        if mixed_k:       # the sweep over a fixed draft length: the 64 regions alone
            return I.mixed_workload(seed=I.BASE_SEED + 4 + 1000 * rank, fixed_draft_len=mixed_k, with_page_chunks=False,
                                    cfg=cfg), False
        return I.mixed_workload(seed=I.BASE_SEED + 4 + 1000 * rank, cfg=cfg), False
    ctx, k = PAGE_SHAPES[name]
    rng = np.random.Generator(np.random.PCG64(I.BASE_SEED + 2 + 1000 * rank))
    emb = I.bf16_round(rng.standard_normal((ctx, cfg.d_model), dtype=np.float32))
    seq = I.SeqInput(emb, np.full(ctx, -1, np.int32), k, k, rng.integers(0, cfg.vocab, size=k, dtype=np.int32), True)
    return I.Workload(name, cfg, I.BASE_SEED + 2, [seq], chunk_len=k), False


_WEIGHTS = {}


def decoder_weights():
    """The 24-layer decoder's seeded weights (host copy, made once per process: both arms read the same values)."""
    if "w" not in _WEIGHTS:
        _WEIGHTS["w"] = I.make_weights(I.DECODER, I.BASE_SEED + 1)
    return _WEIGHTS["w"]


def build_model(flags=0, name="region"):
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = workload_cfg(name)
    weights = decoder_weights() if cfg is I.DECODER else I.make_weights(cfg, I.BASE_SEED + 6)
    return R.DeviceModel(cfg, weights, flags, f"cuda:{torch.cuda.current_device()}")


def plant_along_verify_rows(eng, kv, seqs, first, prefix_lens, cfg, max_rounds=600):
    """Drafts whose first `agree_len` tokens are exactly what a verify call over the whole batch takes for its row
    argmaxes.  The one-token greedy decode is only the first guess: on near-tie rows a many-row call can pick the other
    token (other tile shapes), and everything after such a row then differs.  So the guess is corrected by the call's
    own teacher-forced rows until every sequence is accepted as far as its planted length; then the planted mismatch
    and the random tail go in.  `eng` must run on a context with HSD_FLAG_DETERMINISTIC (bit-reproducible calls)."""
    import torch
    S = len(seqs)
    need = [min(s.agree_len + 1, s.draft_len) for s in seqs]
    cu1 = eng._i32(np.arange(S + 1))
    out1 = eng.alloc_outputs(S, 1, S)
    pending = first.clone()
    hist = []
    for _ in range(max(need)):
        eng.verify_regions(pending, cu1, 1, S, out=out1)
        eng.commit(out1["accept_len"])
        pending = out1["emit_tokens"][:, 0].clone()
        hist.append(pending)
    eng.check_device("greedy continuation")
    kv.seq_lens.copy_(prefix_lens)
    greedy = torch.stack(hist, 1).cpu().numpy() if hist else np.zeros((S, 0), np.int32)
    guess = [np.asarray(greedy[i, :s.draft_len], np.int32).copy() for i, s in enumerate(seqs)]
    for i, s in enumerate(seqs):          # pad to the draft length (the tail is replaced below)
        if len(guess[i]) < s.draft_len:
            guess[i] = np.concatenate([guess[i], s.rand_tokens[len(guess[i]):s.draft_len]]).astype(np.int32)
    f = first.cpu().numpy()
    ks = [s.draft_len for s in seqs]
    T, max_q = sum(ks) + S, max(ks) + 1
    out = eng.alloc_outputs(S, max_q, T)
    rounds = 0
    for rounds in range(max_rounds):
        toks, cu = I.pack_queries(f, guess)
        eng.verify_regions(eng._i32(toks), eng._i32(cu), max_q, T, out=out)
        acc = out["accept_len"].cpu().numpy()
        am = out["row_argmax"].cpu().numpy()
        done = True
        for i, s in enumerate(seqs):
            a = int(acc[i])
            if a < min(s.agree_len, s.draft_len):     # row a's argmax is what the call would have accepted there
                guess[i][a] = am[cu[i] + a]
                done = False
        if done:
            break
    eng.check_device("draft planting")
    drafts = []
    for i, s in enumerate(seqs):
        g = guess[i].copy()
        if s.agree_len < s.draft_len:       # the token the call takes at the planted position: the draft must differ from it
            g[s.agree_len] = am[cu[i] + s.agree_len]
        drafts.append(I.plant_draft(g, s.draft_len, s.agree_len, s.rand_tokens, cfg.vocab, False))
    return drafts, rounds + 1


def build_gpu_state(name, model, rank, world=1, sharded=False, mixed_k=0, random_drafts=False):
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = workload_cfg(name)
    wl, plant = make_workload(name, rank, world, sharded, mixed_k)
    plant = plant and not random_drafts
    seqs = wl.seqs
    S = len(seqs)
    tree = name == "tree"
    kv = R.KvCache(model, [s.prefix_len + s.draft_len + 2 + (2 * WINDOW_N if tree else 0) for s in seqs], seed=wl.seed)
    ks = [s.draft_len for s in seqs]
    total_q = sum(ks) + S
    total_prefix = sum(s.prefix_len for s in seqs)
    eng = R.Engine(model, kv, max(total_prefix, 2 * total_q if tree else total_q), S)
    first = eng.prefill([s.prefix_embeds for s in seqs], [s.prefix_ids for s in seqs])
    eng.check_device("prefill")
    prefix_lens = kv.seq_lens.clone()
    plant_rounds = 0
    accept_det = None
    dsv = None
    if tree:
        # The region's text = the library's own greedy continuation; its first WINDOW_N tokens count as accepted (their
        # K/V rows are written by the one-token steps), the rest is what the two "pipeline drafts" try to predict:
        # copies of the text with substitution errors, the first one where the workload plants its disagreement.
        # Matching the window against them gives two candidates that share a prefix.
        cu1 = eng._i32(np.arange(S + 1))
        out1 = eng.alloc_outputs(S, 1, S)
        pending, hist = first.clone(), []
        for _ in range(TREE_NODES + WINDOW_N):
            eng.verify_regions(pending, cu1, 1, S, out=out1)
            eng.commit(out1["accept_len"])
            pending = out1["emit_tokens"][:, 0].clone()
            hist.append(pending)
        eng.check_device("greedy continuation")
        greedy = torch.stack(hist, 1).cpu().numpy()
        f = first.cpu().numpy()
        texts = [np.concatenate([[f[i]], greedy[i]]).astype(np.int32) for i in range(S)]
        d_list, off, soff = [], [0], [0]
        for i, s in enumerate(seqs):
            a_, b_ = texts[i].copy(), texts[i].copy()
            e1 = min(WINDOW_N + s.agree_len, len(a_) - 1)
            a_[e1] = (a_[e1] + 1) % cfg.vocab
            e2 = min(WINDOW_N + max(1, s.agree_len // 2), len(b_) - 1)
            b_[e2] = (b_[e2] + 2) % cfg.vocab
            for d_ in (a_, b_):
                d_list.append(d_)
                off.append(off[-1] + len(d_))
            soff.append(len(off) - 1)
        prefix_lens = prefix_lens + (WINDOW_N - 1)
        kv.seq_lens.copy_(prefix_lens)
        dsv = dict(window=np.stack([t[:WINDOW_N] for t in texts]).astype(np.int32), tokens=np.concatenate(d_list),
                   off=np.asarray(off, np.int32), soff=np.asarray(soff, np.int32))
        drafts = [np.zeros(TREE_NODES, np.int32) for _ in seqs]     # shapes only: the device packs the rows
    elif plant:
        # Random-weight decoders have near-tie logits on about half their rows, and K slices that add in arrival order
        # flip a per-cent or so of the rows from one call to the next: what a draft "agrees" with is only defined on a
        # context with a fixed summation order.  The drafts are planted there (same weights, same KV cache).
        from paper_2602_12957_b200 import binding as B
        det = model.sibling(B.HSD_FLAG_DETERMINISTIC)
        det_eng = R.Engine(det, kv, total_q, S)
        drafts, plant_rounds = plant_along_verify_rows(det_eng, kv, seqs, first, prefix_lens, cfg)
        toks_d, cu_d = I.pack_queries(first.cpu().numpy(), drafts)
        out_d = det_eng.verify_regions(det_eng._i32(toks_d), det_eng._i32(cu_d), max(ks) + 1, total_q)
        accept_det = float(np.mean([a / k for a, k in zip(out_d["accept_len"].cpu().numpy().tolist(), ks)]))
        del det_eng
        det.close()
    else:
        drafts = [s.rand_tokens[:s.draft_len] for s in seqs]
    toks, cu = I.pack_queries(first.cpu().numpy(), drafts)
    return dict(name=name, cfg=cfg, wl=wl, model=model, kv=kv, eng=eng, toks=toks, cu=cu, total_q=total_q,
                max_q=max(ks) + 1, prefix_lens=prefix_lens, ks=ks, S=S, drafts=drafts, dsv=dsv, planted=plant,
                plant_rounds=plant_rounds, accept_det=accept_det)


def kernel_work_table(cfg, work: RF.StepWork, T: int, lm_rows: int):
    """Algorithmic (flops, bytes) per launch of each kernel class."""
    d, f, V = cfg.d_model, cfg.d_ffn, cfg.vocab
    L = cfg.n_layers
    t = {}
    t["gemm_qkv"] = RF.gemm_work(T, cfg.qkv_out, d)
    t["gemm_o"] = RF.gemm_work(T, d, cfg.n_heads * cfg.head_dim, 8.0)          # fp32 read-modify-write
    t["gemm_gate_up"] = (2.0 * T * 2 * f * d, 2.0 * (T * d + 2 * f * d) + 2.0 * T * f)
    t["gemm_down"] = RF.gemm_work(T, d, f, 8.0)
    t["lm_head_argmax"] = (2.0 * lm_rows * V * d, 2.0 * (lm_rows * d + V * d) + 12.0 * lm_rows)
    t["attention"] = (work.attn_flops / L, work.kv_read_bytes / L + 4.0 * T * cfg.n_heads * cfg.head_dim)
    t["rmsnorm"] = (0.0, 6.0 * T * d)
    return t


class Runner:
    """One workload on the device: the step closure, its CUDA graph, timing and per-kernel profiling."""

    def __init__(self, st, stream, use_graph=True, warmup=3):
        import torch
        from paper_2602_12957_b200 import binding as B
        self.st, self.stream, self.B, self.torch = st, stream, B, torch
        eng, kv = st["eng"], st["kv"]
        dev = eng.dev
        S, T, max_q = st["S"], st["total_q"], st["max_q"]
        self.d_toks, self.d_cu = eng._i32(st["toks"]), eng._i32(st["cu"])
        self.out = eng.alloc_outputs(S, max_q, T)
        self.tree = st["dsv"] is not None
        self.page = st["name"] in PAGE_SHAPES
        if self.tree:
            dsv = st["dsv"]
            self.d_window = eng._i32(dsv["window"])
            self.d_dtok, self.d_doff, self.d_dsoff = eng._i32(dsv["tokens"]), eng._i32(dsv["off"]), eng._i32(dsv["soff"])
            i32 = lambda *shape: torch.empty(*shape, dtype=torch.int32, device=dev)
            self.bout = {"q_tokens": i32(T), "parent": i32(T), "cu_q": i32(S + 1), "n_rows": i32(S)}
            self.out["accept_rows"] = torch.zeros(S, max_q, dtype=torch.int32, device=dev)
            self.out["row_zchild"] = self.out.pop("row_zdraft")
        if self.page:
            self.d_pending = self.d_toks[:1].clone()
            self.d_chunk = self.d_toks[1:].clone()
        ctx = eng.model.ctx
        launches0 = B.hsd_launch_count(ctx)
        with torch.cuda.stream(stream):
            for _ in range(max(3, warmup)):
                self.step()
            stream.synchronize()
            eng.check_device("warmup")
            self.launches_per_step = (B.hsd_launch_count(ctx) - launches0) // max(3, warmup)
            self.graph = None
            if use_graph:
                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, stream=stream):
                    self.step()
                for _ in range(3):
                    self.graph.replay()
                stream.synchronize()

    def step(self):
        st, eng, out = self.st, self.st["eng"], self.out
        if self.tree:
            eng.dsv_build(self.d_window, self.d_dtok, self.d_doff, self.d_dsoff, st["max_q"], out=self.bout)
            eng.verify_tree(self.bout["q_tokens"], self.bout["cu_q"], self.bout["parent"], st["max_q"], st["total_q"],
                            out=out, log_tau=LOG_TAU_TREE)
            eng.commit_tree(out["accept_len"], out["accept_rows"])
        elif self.page:      # Stage 2 goes through its own entry point
            eng.verify_page(0, self.d_pending, self.d_chunk, out=out)
            eng.commit(out["accept_len"])
        else:
            eng.verify_regions(self.d_toks, self.d_cu, st["max_q"], st["total_q"], out=out)
            eng.commit(out["accept_len"])
        st["kv"].seq_lens.copy_(st["prefix_lens"])          # rewind so every timed step sees the same state

    def run(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.step()

    def timed(self, steps, barrier, uuid, min_seconds=0.0):
        """(ms per step, clocks, steps run): `steps` replays (more, up to min_seconds of work, when asked) between two
        CUDA events on the launching stream, clocks sampled meanwhile."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if min_seconds > 0:
            with torch.cuda.stream(self.stream):
                p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                p0.record(self.stream)
                for _ in range(3):
                    self.run()
                p1.record(self.stream)
                self.stream.synchronize()
            steps = max(steps, int(min_seconds * 1e3 / max(1e-3, p0.elapsed_time(p1) / 3)))
        sampler = ClockSampler(uuid)
        with torch.cuda.stream(self.stream):
            barrier()
            torch.cuda.cudart().cudaProfilerStart()       # lets `ncu --profile-from-start off` see the timed steps only
            e0.record(self.stream)
            for _ in range(steps):
                self.run()
            e1.record(self.stream)
            barrier()
            torch.cuda.cudart().cudaProfilerStop()
        ms = e0.elapsed_time(e1) / steps
        clocks = sampler.stop()
        clocks["sampled"] = "timed region"
        return ms, clocks, steps

    def per_step_stats(self, n=50):
        """Median and minimum over `n` replays timed one by one (an event pair around each), in a pass of its own."""
        torch = self.torch
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        with torch.cuda.stream(self.stream):
            for _ in range(3):
                self.run()
            evs[0].record(self.stream)
            for i in range(n):
                self.run()
                evs[i + 1].record(self.stream)
            self.stream.synchronize()
        t = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(n))
        return {"median": t[n // 2], "min": t[0], "replays": n}

    def draft_tokens(self):
        if self.tree:          # the nodes the device actually packed
            return int(self.bout["n_rows"].sum().item()) - self.st["S"]
        return int(sum(self.st["ks"]))

    def profile(self, prof_steps):
        """Per-kernel-class durations: the same step launched eagerly with a CUDA event right before and right after
        every launch (each interval owns both its ends; kernels do not overlap across an event)."""
        B, torch = self.B, self.torch
        ctx = self.st["eng"].model.ctx
        with torch.cuda.stream(self.stream):
            B.hsd_profile_enable(ctx, 1)
            for _ in range(prof_steps):
                self.step()
            self.stream.synchronize()
            _, prof = B.hsd_profile_read(ctx)
            B.hsd_profile_enable(ctx, 0)
        return prof


def two_stage_workload(device, seed=I.BASE_SEED + 5, mean_run=16.0, n_lanes=8):
    """One synthetic page through the whole hierarchy (Sec. 3.1): Stage 1 on the region workload's 16 crops (each
    region's output as long as its configured draft + 1) on `n_lanes` lanes with continuous hand-over; aggregation
    (Eq. 3); Stage 2 on a page prefix of 4096 visual rows + 256 prompt tokens against the aggregated Stage-1 outputs
    themselves.  The decoder is the chain decoder of `inputs.make_chain_weights` (same architecture and kernel work
    as the timed decoder, but its greedy text is known and decided by wide margins): the last prompt token of every
    crop is chosen so that the page's text is the concatenation of the regions' texts, which is the structure the
    method relies on.  The "pipeline drafts" of Stage 1 are two copies of each region's text with substitution errors
    every `mean_run` tokens on average (geometric), damaged independently."""
    import torch
    from paper_2602_12957_b200 import driver as DR
    from paper_2602_12957_b200 import runtime as R
    cfg = I.DECODER
    if "chain" not in _WEIGHTS:
        _WEIGHTS["chain"] = I.make_chain_weights(cfg, I.BASE_SEED + 1)
    weights, order = _WEIGHTS["chain"]
    model = R.DeviceModel(cfg, weights, 0, device)
    wl = I.region_workload(seed=I.BASE_SEED + 1, cfg=cfg)
    pw = I.page_workload(cfg=cfg)
    lengths = [s.draft_len + 1 for s in wl.seqs]
    page_len = int(sum(lengths))
    offs = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    p0 = 12345
    walk = lambda start, n: order[(start + 1 + np.arange(n)) % cfg.vocab].astype(np.int32)

    def with_last_prompt_token(seq, pos):
        ids = seq.prefix_ids.copy()
        ids[-1] = order[pos % cfg.vocab]
        return (seq.prefix_embeds, ids)
    regions = [with_last_prompt_token(s_, p0 + int(offs[i])) for i, s_ in enumerate(wl.seqs)]
    page = with_last_prompt_token(pw.seqs[0], p0)
    texts = [walk(p0 + int(offs[i]), lengths[i]) for i in range(len(regions))]
    page_text = walk(p0, page_len)
    rng = np.random.Generator(np.random.PCG64(seed))

    def damaged(t):
        d = np.asarray(t, np.int64).copy()
        pos = 3 + int(rng.geometric(1.0 / mean_run))
        while pos < len(d):
            d[pos] = (d[pos] + 1 + int(rng.integers(0, cfg.vocab - 1))) % cfg.vocab
            pos += int(rng.geometric(1.0 / mean_run))
        return d.astype(np.int32)
    region_drafts = [[damaged(t), damaged(t)] for t in texts]
    run = DR.run_page(model, regions, region_drafts, lengths, page, page_len, n_lanes=n_lanes, log_tau=LOG_TAU_TREE,
                      seed=seed)
    s1, s2 = run.stage1, run.stage2
    ok1 = all(np.array_equal(a, b) for a, b in zip(s1.tokens, texts))
    ok2 = np.array_equal(s2.tokens[0], page_text)
    ok_draft = all(np.array_equal(a, b) for a, b in zip(run.page_draft, texts))
    model.close()
    tok1, tok2 = int(sum(len(t) for t in s1.tokens)), int(len(s2.tokens[0]))
    decode_ms = s1.ms + run.aggregate_ms + s2.ms
    return {"workload": two_stage_workload.__doc__.split("\n")[0].strip() + " tau 0.75, window 3, 128 packed rows per sequence",
            "decoder": "chain decoder: the timed decoder's architecture with residual branches scaled by 0.004 and an LM "
                       "head built from the embedding table, so that its greedy text is a known walk with logit margins "
                       "near 70; random-init weights give half the rows a top-1/top-2 gap below 0.1 and a text that "
                       "changes with a kernel's summation order",
            "outputs_equal_the_known_texts": {"stage1": bool(ok1), "page_draft": bool(ok_draft), "stage2": bool(ok2)},
            "prefill_ms": run.prefill_ms, "stage1_ms": s1.ms, "aggregate_ms": run.aggregate_ms, "stage2_ms": s2.ms,
            "decode_ms": decode_ms, "tokens_per_page": tok1 + tok2, "tokens_per_s": (tok1 + tok2) / (decode_ms * 1e-3),
            "stage1": {"regions": len(regions), "lanes": n_lanes, "tokens": tok1, "batch_steps": s1.batch_steps,
                       "sequence_steps": int(s1.steps.sum()), "aal": s1.aal, "ms_per_batch_step": s1.ms / max(1, s1.batch_steps),
                       "drafts": f"two copies of each region's text, substitution errors every {mean_run:g} tokens on average"},
            "stage2": {"tokens": tok2, "steps": int(s2.steps.sum()), "aal": s2.aal,
                       "ms_per_step": s2.ms / max(1, s2.batch_steps), "drafts": "the aggregated Stage-1 outputs (Eq. 3)"},
            "launch": "CUDA graph of 8 steps between two reads of the device's not-finished counter"}


def choose_peak(peaks, clocks):
    """The bf16 denominator: the burst figure when the SM clock held >= 0.95 of its maximum during the timed region
    (the burst measurement's own condition), else the sustained, power-capped figure."""
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if sm and mx and sm >= 0.95 * mx:
        return peaks["bf16_tflops"], "burst"
    return peaks["bf16_tflops_sustained"], "sustained"


def roofline_report(st, prof, prof_steps, ms_step, clocks, peaks, peak_src, traffic_table=None):
    cfg = st["cfg"]
    T = st["total_q"]
    tree = st["dsv"] is not None
    ctx_lens = [int(x) for x in st["prefix_lens"].cpu().numpy().tolist()]
    work = RF.step_work(cfg, ctx_lens, [k + 1 for k in st["ks"]])
    table = kernel_work_table(cfg, work, T, 2 * T if tree else T)
    tot_ms = sum(v[0] for v in prof.values()) or 1.0
    kernels = {k: {"ms_per_step": v[0] / prof_steps, "launches_per_step": v[1] / prof_steps,
                   "share": v[0] / tot_ms} for k, v in prof.items()}
    bw = peaks["hbm_gbs"] * 1e9
    pk_tf, pk_kind = choose_peak(peaks, clocks)
    pk = pk_tf * 1e12

    def dur_of(k):      # seconds per launch; the LM-head class has one GEMM per step beside two tiny kernels
        return prof[k][0] * 1e-3 / (prof_steps if k == "lm_head_argmax" else prof[k][1])

    # the dominant kernel class: the largest measured total; classes within 10 % of it count as tied (on the region batch
    # attention and gate/up are 22 % each and trade places from run to run) and the tie goes to the one whose algorithmic
    # roofline time is larger; every class's own fraction is in `kernels`
    cands = [k for k in prof if k in table]
    t_max = max(prof[k][0] for k in cands)

    def roof_time(k):
        fl, nb = table[k]
        return max(fl / pk, nb / bw) * prof[k][1]
    top = max((k for k in cands if prof[k][0] >= 0.90 * t_max), key=roof_time)
    flops, nbytes = table[top]
    dur = dur_of(top)
    if flops / pk >= nbytes / bw:
        roof = {"kernel": top, "bound": "tensor", "achieved": flops / dur / 1e12, "peak": pk_tf, "unit": "TFLOP/s",
                "frac_of_burst": flops / dur / 1e12 / peaks["bf16_tflops"],
                "frac_of_sustained": flops / dur / 1e12 / peaks["bf16_tflops_sustained"]}
        roof["peak_source"] = (f"{peak_src} bf16 {pk_kind} figure (SM clock median {clocks.get('sm_mhz')} of "
                               f"{clocks.get('sm_max_mhz')} MHz during the timed region)")
    else:
        roof = {"kernel": top, "bound": "hbm", "achieved": nbytes / dur / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "peak_source": f"{peak_src} (STREAM-style copy bandwidth)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = (traffic_table or {}).get(top)
    roof["us_per_launch"] = dur * 1e6
    roof["timing"] = ("CUDA events right before and after every launch of an eagerly launched step (each interval owns "
                      "both ends, no overlap between kernels); the timed step itself is a CUDA graph whose kernels "
                      "overlap through programmatic dependent launch, so the intervals sum to more than the step")
    for k, (fl, nb) in table.items():
        if k in prof and prof[k][1] > 0:
            d_k = dur_of(k)
            tensor_k = fl / pk >= nb / bw
            kernels[k]["bound"] = "tensor" if tensor_k else "hbm"
            kernels[k]["roofline_frac"] = (fl / d_k / pk) if tensor_k else (nb / d_k / bw)
    t_roof = RF.roofline_time(work.bytes, work.flops, bw, pk)
    tensor_step = work.flops / pk > work.bytes / bw
    step_roof = {"roofline_us": t_roof * 1e6, "frac": t_roof / (ms_step * 1e-3), "bytes": work.bytes, "flops": work.flops,
                 "bound": "tensor" if tensor_step else "hbm", "bf16_peak": pk_kind,
                 "frac_of_burst": RF.roofline_time(work.bytes, work.flops, bw, peaks["bf16_tflops"] * 1e12) / (ms_step * 1e-3),
                 "frac_of_sustained": RF.roofline_time(work.bytes, work.flops, bw,
                                                       peaks["bf16_tflops_sustained"] * 1e12) / (ms_step * 1e-3),
                 "sum_of_kernel_intervals_ms": tot_ms / prof_steps}
    return roof, step_roof, kernels, ctx_lens


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2602_12957_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    model = build_model(args.flags, args.workload)
    st = build_gpu_state(args.workload, model, rank, world, args.sharded, args.mixed_k, args.random_drafts)
    eng, kv, cfg = st["eng"], st["kv"], st["cfg"]
    dev = eng.dev
    S, T, max_q = st["S"], st["total_q"], st["max_q"]
    stream = torch.cuda.Stream(device=dev)
    runner = Runner(st, stream, use_graph=not args.no_graph, warmup=args.warmup)
    tree = runner.tree

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    ms_step, clocks, _ = runner.timed(args.steps, barrier, uuid)
    one_by_one = runner.per_step_stats(100)
    if clocks["samples"] < 3:        # a short timed region leaves nvidia-smi nothing to sample: replay longer
        sampler = ClockSampler(uuid)
        with torch.cuda.stream(stream):
            t_end = time.time() + 1.5
            while time.time() < t_end:
                for _ in range(20):
                    runner.run()
                stream.synchronize()
        clocks = sampler.stop()
        clocks["sampled"] = "1.5 s replay of the same step after the timed region"
    if world > 1:
        tt = torch.tensor([ms_step], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_step = float(tt.item())
    draft_tokens = runner.draft_tokens()
    all_tokens = draft_tokens
    if world > 1:
        tt = torch.tensor([float(draft_tokens)], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.SUM)
        all_tokens = float(tt.item())
    value = all_tokens / (ms_step * 1e-3)

    # ---- end to end through the C-ABI call that takes HOST buffers (pinned): every step copies the packed drafts
    # host->device, runs verify + commit, copies accept_len / n_emit / emitted tokens device->host and synchronises
    h_toks = torch.from_numpy(st["toks"]).pin_memory()
    h_cu = torch.from_numpy(st["cu"]).pin_memory()
    h_acc = torch.empty(S, dtype=torch.int32).pin_memory()
    h_nem = torch.empty(S, dtype=torch.int32).pin_memory()
    h_emit = torch.empty(S, max_q, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(args.steps, 200))
    ctx = eng.model.ctx
    h_win = torch.from_numpy(st["dsv"]["window"]).pin_memory() if tree else None

    def e2e_step():
        if tree:     # the drafts stay resident (they are fixed per page); per step the window goes in, the results out
            runner.d_window.copy_(h_win, non_blocking=True)
            runner.step()
            h_acc.copy_(runner.out["accept_len"], non_blocking=True)
            h_nem.copy_(runner.out["n_emit"], non_blocking=True)
            h_emit.copy_(runner.out["emit_tokens"], non_blocking=True)
            stream.synchronize()
        else:
            rc, _ = B.hsd_verify_regions_host(ctx, kv.c, S, h_cu, h_toks, None, 0.0, 1, h_acc, h_emit, h_nem, eng.ws.ptr,
                                              eng.ws.bytes, stream.cuda_stream)
            B.check(rc, "hsd_verify_regions_host")
            kv.seq_lens.copy_(st["prefix_lens"])          # rewind (bench artefact: every step sees the same state)

    with torch.cuda.stream(stream):
        for _ in range(3):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        stream.synchronize()
        t1 = time.perf_counter()
        barrier()
    e2e_ms = (t1 - t0) * 1e3 / e2e_steps
    if world > 1:
        tt = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        e2e_ms = float(tt.item())
    e2e = {"value": all_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": int(h_win.numel() * 4 if tree else h_toks.numel() * 4 + h_cu.numel() * 4),
           "d2h_bytes_per_step": int((h_acc.numel() + h_nem.numel() + h_emit.numel()) * 4 + 16),
           "call": "hsd_verify_regions_host (pinned host buffers; the library replays the step as a CUDA graph it captured "
                   "at the second call of this shape; stream synchronised per step)" if not tree else
                   "hsd_dsv_build + hsd_verify_tree + hsd_kv_commit_tree (eager launches), the window copied in from and "
                   "the results out to pinned host memory on the same stream, synchronised per step"}
    accept_mean = float(np.mean([a / k for a, k in zip(h_acc.numpy().tolist(), st["ks"])]))

    peaks, peak_src = load_peaks()
    prof_steps = max(3, min(args.steps, 30))
    prof = runner.profile(prof_steps)
    roof, step_roof, kernels, ctx_lens = roofline_report(st, prof, prof_steps, ms_step, clocks, peaks, peak_src,
                                                         NCU_TRAFFIC_BYTES.get(args.workload))

    # ---- one step of every other configuration (one GPU only; the other ranks would only repeat it)
    extra = {}
    launches_per_step = int(runner.launches_per_step)
    if world == 1 and args.workload == "region" and not args.only_region:
        del runner
        for name in EXTRA_WORKLOADS:
            model2 = model
            if workload_cfg(name) is not I.DECODER:
                model2 = build_model(0, name)
            st2 = build_gpu_state(name, model2, 0)
            r2 = Runner(st2, stream, use_graph=not args.no_graph, warmup=3)
            ms2, clk2, n2 = r2.timed(20, barrier, uuid, min_seconds=1.0)
            pr2 = r2.profile(5)
            roof2, sroof2, kern2, ctx2 = roofline_report(st2, pr2, 5, ms2, clk2, peaks, peak_src, NCU_TRAFFIC_BYTES.get(name))
            tok2 = r2.draft_tokens()
            extra[name] = {"workload": WORKLOADS[name], "ms_per_step": ms2, "steps": n2, "tokens_per_s": tok2 / (ms2 * 1e-3),
                           "ms_per_step_one_by_one": r2.per_step_stats(),
                           "draft_tokens": tok2, "query_rows": st2["total_q"], "context_tokens": int(sum(ctx2)),
                           "launches_per_step": int(r2.launches_per_step),
                           "step_roofline_frac": sroof2["frac"], "step_roofline_frac_of_burst": sroof2["frac_of_burst"],
                           "step_roofline_frac_of_sustained": sroof2["frac_of_sustained"], "step_bound": sroof2["bound"],
                           "top_kernel": roof2["kernel"], "top_kernel_bound": roof2["bound"],
                           "top_kernel_frac": roof2["frac"], "top_kernel_us": roof2["us_per_launch"],
                           "top_kernel_traffic": roof2["traffic"], "clocks": clk2,
                           "kernels": {k: {"ms_per_step": round(v["ms_per_step"], 4),
                                           "roofline_frac": round(v.get("roofline_frac", 0.0), 3)} for k, v in kern2.items()}}
            if not args.no_cpu_baseline and name not in ("tree", "region_hd128"):   # (the oracle's tree form and the second decoder are not timed)
                extra[name]["cpu_baseline"] = cpu_baseline_sample(st2["wl"], ctx2, budget_s=6.0, steps=1, max_rows=128)
            del r2, st2
            if model2 is not model:
                model2.close()
            del model2
            torch.cuda.empty_cache()
        with torch.cuda.stream(stream):
            extra["two_stage"] = two_stage_workload(f"cuda:{torch.cuda.current_device()}")
        torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_sample(st["wl"], ctx_lens, budget_s=25.0, steps=3)
        if args.workload == "region" and not args.only_region:
            cpu["tiny"] = tiny_both_arms(stream)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(3, args.warmup), "ms_per_step": ms_step, "ms_per_step_one_by_one": one_by_one,
                "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOADS[args.workload] + (f" [64 regions only, every draft {args.mixed_k} tokens]"
                                                                   if args.workload == "mixed" and args.mixed_k else ""),
                           "regions_per_gpu": S, "query_rows_per_gpu": T, "draft_tokens_per_gpu": draft_tokens,
                           "context_tokens_per_gpu": int(sum(ctx_lens)),
                           "mean_acceptance_rate": st["accept_det"] if st["accept_det"] is not None else accept_mean,
                           "mean_acceptance_rate_timed_context": accept_mean,
                           "planted_acceptance_rate": float(np.mean([s.agree_len / s.draft_len for s in st["wl"].seqs])),
                           "drafts": ("planted along the row argmaxes of the whole-batch verify call on a context with a "
                                      f"fixed summation order ({st['plant_rounds']} correction rounds after the one-token "
                                      "greedy decode), where the call accepts exactly the planted lengths; the timed "
                                      "context adds its K slices in arrival order, which flips near-tie rows (random "
                                      "weights: half the rows have a top-1/top-2 gap below 0.1) and shortens what it accepts"
                                      if st["planted"] else "random tokens (kernel time does not depend on token values)"),
                           "l2_policy": "inputs larger than L2: 822 MB of weights are streamed every step",
                           "launch": "CUDA graph replay" if not args.no_graph else "eager",
                           "sharding": ("one batch of 16 x N regions split across ranks by the cost model, "
                                        if args.sharded else "16 regions per rank, ") + "no data-path collective"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "gpu_launches_per_step": launches_per_step, "roofline": roof, "step_roofline": step_roof, "kernels": kernels, "workloads": extra, "cpu_baseline": cpu}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------ oracle arm
def cpu_baseline_sample(wl, ctx_lens, budget_s=25.0, steps=3, warmup=0, max_rows=None):
    """Times the oracle (float32 numpy, as it stands) on one verify step of the workload's sequences, cheapest first,
    as many as one step's budget allows.  The cached K/V of the context rows is filled with random values of the right
    shape instead of an oracle prefill (untimed either way; the step's time does not depend on the values).  With
    max_rows only the first max_rows - 1 draft tokens of every sequence are verified (long chunks)."""
    from oracle import hsd_oracle as O
    cfg = wl.cfg
    model = O.Decoder(cfg, decoder_weights(), np.float32)
    rng = np.random.default_rng(0)
    order = sorted(range(len(wl.seqs)), key=lambda i: ctx_lens[i] * (wl.seqs[i].draft_len + 1))

    def make(i):
        c = O.CachedSequence(model)
        shape = (int(ctx_lens[i]), cfg.n_kv_heads, cfg.head_dim)
        c.k = [rng.standard_normal(shape, dtype=np.float32) for _ in range(cfg.n_layers)]
        c.v = [rng.standard_normal(shape, dtype=np.float32) for _ in range(cfg.n_layers)]
        k = wl.seqs[i].draft_len if max_rows is None else min(wl.seqs[i].draft_len, max_rows - 1)
        return c, int(rng.integers(0, cfg.vocab)), wl.seqs[i].rand_tokens[:k]

    # grow the sample while one step fits the budget (first sequence always taken)
    caches, pend, drafts, used, t_one = [], [], [], [], 0.0
    for i in order:
        c, p, d = make(i)
        t0 = time.perf_counter()
        O.verify_regions(model, [c], [p], [d])
        dt = time.perf_counter() - t0
        if used and (t_one + dt) * (steps + warmup) > budget_s:
            break
        caches.append(c); pend.append(p); drafts.append(d); used.append(i)
        t_one += dt
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        O.verify_regions(model, caches, pend, drafts)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    k = int(sum(len(d) for d in drafts))
    t = float(np.mean(times))
    whole = len(used) == len(wl.seqs) and max_rows is None
    return {"value": k / t, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": (f"{'all' if whole else len(used)} of {len(wl.seqs)} sequences of the {wl.name} workload"
                       f"{'' if whole else ' (cheapest first)'}: {k} draft tokens over {int(sum(ctx_lens[i] for i in used))} "
                       f"context tokens" + (f", first {max_rows} rows of every chunk" if max_rows else "") +
                       f"; float32 numpy oracle, context K/V prefilled with random values (untimed), "
                       f"{len(times)} timed step(s), threads as numpy's BLAS takes them"),
            "ms_per_step": t * 1e3, "steps": len(times)}


def tiny_both_arms(stream):
    """The Tiny configuration (1 layer, d 256, 4 regions x (128-token prefix + 16-token draft)): one verify step on
    the GPU (graph replay) and in the float64 oracle."""
    import torch
    from oracle import hsd_oracle as O
    from paper_2602_12957_b200 import runtime as R
    wl = I.tiny_workload()
    weights = I.make_weights(wl.cfg, wl.seed)
    model = O.Decoder(wl.cfg, weights, np.float64)
    caches, pend, drafts = [], [], []
    for s in wl.seqs:
        c = O.CachedSequence(model)
        pend.append(c.prefill(s.prefix_embeds, s.prefix_ids))
        caches.append(c)
        drafts.append(s.rand_tokens[:s.draft_len])
    t0 = time.perf_counter()
    for _ in range(3):
        O.verify_regions(model, caches, pend, drafts)
    cpu_ms = (time.perf_counter() - t0) * 1e3 / 3
    dm = R.DeviceModel(wl.cfg, weights, 0)
    kv = R.KvCache(dm, [s.prefix_len + s.draft_len + 2 for s in wl.seqs], seed=wl.seed)
    S, T = len(wl.seqs), sum(s.draft_len + 1 for s in wl.seqs)
    eng = R.Engine(dm, kv, max(sum(s.prefix_len for s in wl.seqs), T), S)
    eng.prefill([s.prefix_embeds for s in wl.seqs], [s.prefix_ids for s in wl.seqs])
    lens = kv.seq_lens.clone()
    toks, cu = I.pack_queries(pend, drafts)
    d_t, d_c = eng._i32(toks), eng._i32(cu)
    out = eng.alloc_outputs(S, 17, T)

    def step():
        eng.verify_regions(d_t, d_c, 17, T, out=out)
        eng.commit(out["accept_len"])
        kv.seq_lens.copy_(lens)
    with torch.cuda.stream(stream):
        for _ in range(3):
            step()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(200):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    k = sum(len(d) for d in drafts)
    gpu_ms = e0.elapsed_time(e1) / 200
    return {"workload": "Tiny verify: 1 layer, d 256, 4 regions x (128-token prefix, 16-token draft)",
            "gpu_us_per_step": gpu_ms * 1e3, "gpu_tokens_per_s": k / (gpu_ms * 1e-3),
            "oracle_ms_per_step": cpu_ms, "oracle_tokens_per_s": k / (cpu_ms * 1e-3), "oracle": "float64 numpy, all 4 regions"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = I.region_workload(seed=I.BASE_SEED + 1, cfg=I.DECODER)
    ctx = [s.prefix_len for s in wl.seqs]
    r = cpu_baseline_sample(wl, ctx, budget_s=150.0, steps=max(1, args.steps), warmup=max(0, min(args.warmup, 1)))
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": r["steps"], "warmup": max(0, min(args.warmup, 1)),
            "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOADS["region"] + " [bounded sample, see cpu_baseline.sample]"},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def respawn_under_torchrun(args):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node and pass their output on."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")        # the log says which transport and algorithm NCCL chose (stderr)
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-region", action="store_true", help="skip the other configurations' steps (`workloads`)")
    ap.add_argument("--sharded", action="store_true",
                    help="N > 1: one batch of 16 x N regions split across the ranks by the cost model, instead of 16 "
                         "regions drawn per rank")
    ap.add_argument("--workload", default="region", choices=sorted(WORKLOADS),
                    help="region = the benchmark line; the others time one step of the other configurations")
    ap.add_argument("--mixed-k", type=int, default=0,
                    help="with --workload mixed: the 64 regions alone, every draft this many tokens long (the k sweep)")
    ap.add_argument("--flags", type=int, default=0, help="HSD_FLAG_* bits for the context (debugging / ablations)")
    ap.add_argument("--random-drafts", action="store_true",
                    help="skip the pass that plants agreement (for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_torchrun(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
