#!/usr/bin/env python
"""Benchmark of the HSD draft-verification step on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (one process per GPU)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands, on host cores

One step = one pass of the whole hot path over one batch: pack/embed, 24 x (norm, QKV+RoPE+KV write, paged
causal attention, O, norm, gate/up+SwiGLU, down), final norm, LM head + argmax + draft logit, accept/emit,
KV commit.  Workload (default): the region-level stage — 16 regions per GPU, prefixes 256-1024 visual rows,
lognormal draft lengths (mean 64, clipped 8-256), planted agreement with mean acceptance 0.8, paged KV with
64-token blocks and shuffled physical blocks.  Inputs are synthetic and seeded; weights are random-init.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_12957_b200 import inputs as I          # noqa: E402
from paper_2602_12957_b200 import roofline as RF       # noqa: E402

METRIC = "draft tokens verified per second (verify step: forward over paged prefix + accept + KV commit)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic per launch of the dominant kernel classes, from the ncu captures summarised under profiles/
# (dram__bytes_read.sum + dram__bytes_write.sum); None where no capture exists yet.
NCU_TRAFFIC_BYTES = {"attention": 30.96e6, "gemm_gate_up": 19.52e6, "gemm_qkv": 7.28e6, "gemm_o": 10.25e6,
                     "gemm_down": 24.67e6}     # region workload only


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


# ------------------------------------------------------------------------------------------------ workload
WORKLOADS = {
    "region": "region-level stage: 24-layer decoder d1024 16q/8kv x64 ffn4096 vocab32768, 16 regions per GPU, prefix "
              "256-1024, lognormal drafts mean 64 (8-256), acceptance 0.8, paged KV block 64",
    "page": "page-level stage, one chunk mid-schedule: batch 1, 6400 committed tokens, chunk of 512 draft tokens",
    "long1024": "long-document page verify, one chunk mid-schedule: batch 1, 10240 committed tokens, chunk of 1024",
    "long2048": "long-document page verify, one chunk mid-schedule: batch 1, 10240 committed tokens, chunk of 2048",
    "tree": "one step of the decoupled-verification loop on the region batch's 16 prefixes (256-1024): window matching "
            "(n = 3) against two damaged copies of each region's text and prefix-tree packing on the device (128 rows "
            "per sequence), tree verification at tau 0.75, compaction of the accepted path's K/V rows",
    "mixed": "mixed serving batch: 64 regions (prefix 128-2048, lognormal drafts mean 96, 8-512) + 2 page chunks of 1024 "
             "over 4352-token prefixes, one varlen launch",
}


TREE_NODES = 127     # nodes below the root: 128 packed rows per sequence, the paper's packing limit (Sec. 4.3)
TREE_MAIN = 64       # the planted agreement lengths of the region workload are scaled to this many tokens
WINDOW_N = 3         # reference window (Sec. 4.3)
LOG_TAU_TREE = float(np.log(0.75))


def make_workload(args, rank):
    """The seeded workload of this rank.  Region: planted drafts; the others (extra, not the default bench line):
    random drafts, since kernel time does not depend on token values."""
    cfg = I.DECODER
    name = getattr(args, "workload", "region")
    if name == "region":
        return I.region_workload(seed=I.BASE_SEED + 1 + 1000 * rank, cfg=cfg)
    if name == "tree":
        wl = I.region_workload(seed=I.BASE_SEED + 1 + 1000 * rank, cfg=cfg)
        for s_ in wl.seqs:          # same prefixes; the draft becomes a 127-node tree whose main path agrees as planted
            s_.agree_len = int(round(TREE_MAIN * s_.agree_len / max(1, s_.draft_len)))
            s_.draft_len = TREE_NODES
        return wl
    args.random_drafts = True
    if name == "mixed":
        k = getattr(args, "mixed_k", 0)
        if k:       # the sweep over a fixed draft length: the 64 regions alone
            return I.mixed_workload(seed=I.BASE_SEED + 4 + 1000 * rank, fixed_draft_len=k, with_page_chunks=False, cfg=cfg)
        return I.mixed_workload(seed=I.BASE_SEED + 4 + 1000 * rank, cfg=cfg)
    ctx, k = {"page": (6400, 512), "long1024": (10240, 1024), "long2048": (10240, 2048)}[name]
    rng = np.random.Generator(np.random.PCG64(I.BASE_SEED + 2 + 1000 * rank))
    emb = I.bf16_round(rng.standard_normal((ctx, cfg.d_model), dtype=np.float32))
    seq = I.SeqInput(emb, np.full(ctx, -1, np.int32), k, k, rng.integers(0, cfg.vocab, size=k, dtype=np.int32), True)
    return I.Workload(name, cfg, I.BASE_SEED + 2, [seq], chunk_len=k)


def build_gpu_state(args, rank):
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = I.DECODER
    wl = make_workload(args, rank)
    weights = I.make_weights(cfg, I.BASE_SEED + 1)
    model = R.DeviceModel(cfg, weights, getattr(args, "flags", 0), f"cuda:{torch.cuda.current_device()}")
    del weights
    seqs = wl.seqs
    S = len(seqs)
    tree = getattr(args, "workload", "region") == "tree"
    kv = R.KvCache(model, [s.prefix_len + s.draft_len + 2 + (2 * WINDOW_N if tree else 0) for s in seqs], seed=wl.seed)
    ks = [s.draft_len for s in seqs]
    total_q = sum(ks) + S
    total_prefix = sum(s.prefix_len for s in seqs)
    eng = R.Engine(model, kv, max(total_prefix, 2 * total_q if tree else total_q), S)
    first = eng.prefill([s.prefix_embeds for s in seqs], [s.prefix_ids for s in seqs])
    eng.check_device("prefill")
    prefix_lens = kv.seq_lens.clone()

    # greedy continuation by plain one-token steps (empty drafts), to plant the agreement lengths
    need = 0 if args.random_drafts else max(min(s.agree_len + 1, s.draft_len) for s in seqs)
    if tree:
        need = TREE_NODES + WINDOW_N
    cu1 = eng._i32(np.arange(S + 1))
    out1 = eng.alloc_outputs(S, 1, S)
    pending = first.clone()
    hist = []
    for _ in range(need):
        eng.verify_regions(pending, cu1, 1, S, out=out1)
        eng.commit(out1["accept_len"])
        pending = out1["emit_tokens"][:, 0].clone()
        hist.append(pending)
    eng.check_device("greedy continuation")
    greedy = torch.stack(hist, 1).cpu().numpy() if hist else np.zeros((S, 0), np.int32)
    kv.seq_lens.copy_(prefix_lens)
    if tree:
        drafts = []
    elif args.random_drafts:    # profiling runs: kernel time does not depend on token values
        drafts = [s.rand_tokens[:s.draft_len] for s in seqs]
    else:
        drafts = [I.plant_draft(greedy[i], s.draft_len, s.agree_len, s.rand_tokens, cfg.vocab, False)
                  for i, s in enumerate(seqs)]
    dsv = None
    if tree:
        # The region's text = the library's own greedy continuation; its first WINDOW_N tokens count as accepted (their
        # K/V rows were written by the one-token steps above), the rest is what the two "pipeline drafts" try to
        # predict: copies of the text with substitution errors, the first one where the workload plants its
        # disagreement.  Matching the window against them gives two candidates that share a prefix.
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
    toks, cu = I.pack_queries(first.cpu().numpy(), drafts)
    return dict(cfg=cfg, wl=wl, model=model, kv=kv, eng=eng, toks=toks, cu=cu, total_q=total_q, max_q=max(ks) + 1,
                prefix_lens=prefix_lens, ks=ks, S=S, drafts=drafts, dsv=dsv)


def kernel_work_table(cfg, work: RF.StepWork, T: int):
    """Algorithmic (flops, bytes) per launch of each kernel class."""
    d, f, V = cfg.d_model, cfg.d_ffn, cfg.vocab
    L = cfg.n_layers
    t = {}
    t["gemm_qkv"] = RF.gemm_work(T, cfg.qkv_out, d)
    t["gemm_o"] = RF.gemm_work(T, d, cfg.n_heads * cfg.head_dim, 8.0)          # fp32 read-modify-write
    t["gemm_gate_up"] = (2.0 * T * 2 * f * d, 2.0 * (T * d + 2 * f * d) + 2.0 * T * f)
    t["gemm_down"] = RF.gemm_work(T, d, f, 8.0)
    t["lm_head_argmax"] = (2.0 * T * V * d, 2.0 * (T * d + V * d) + 12.0 * T)       # (a tree step runs it over 2T rows)
    t["attention"] = (work.attn_flops / L, work.kv_read_bytes / L + 4.0 * T * cfg.n_heads * cfg.head_dim)
    t["rmsnorm"] = (0.0, 6.0 * T * d)
    return t


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
    st = build_gpu_state(args, rank)
    eng, kv, cfg = st["eng"], st["kv"], st["cfg"]
    dev = eng.dev
    S, T, max_q = st["S"], st["total_q"], st["max_q"]
    d_toks, d_cu = eng._i32(st["toks"]), eng._i32(st["cu"])
    out = eng.alloc_outputs(S, max_q, T)
    stream = torch.cuda.Stream(device=dev)
    tree = st["dsv"] is not None
    if tree:
        dsv = st["dsv"]
        d_window = eng._i32(dsv["window"])
        d_dtok, d_doff, d_dsoff = eng._i32(dsv["tokens"]), eng._i32(dsv["off"]), eng._i32(dsv["soff"])
        i32 = lambda *shape: torch.empty(*shape, dtype=torch.int32, device=dev)
        bout = {"q_tokens": i32(T), "parent": i32(T), "cu_q": i32(S + 1), "n_rows": i32(S)}
        out["accept_rows"] = torch.zeros(S, max_q, dtype=torch.int32, device=dev)
        out["row_zchild"] = out.pop("row_zdraft")

    def step():
        if tree:
            eng.dsv_build(d_window, d_dtok, d_doff, d_dsoff, max_q, out=bout)
            eng.verify_tree(bout["q_tokens"], bout["cu_q"], bout["parent"], max_q, T, out=out, log_tau=LOG_TAU_TREE)
            eng.commit_tree(out["accept_len"], out["accept_rows"])
        else:
            eng.verify_regions(d_toks, d_cu, max_q, T, out=out)
            eng.commit(out["accept_len"])
        kv.seq_lens.copy_(st["prefix_lens"])          # rewind so every timed step sees the same state

    launches0 = B.hsd_launch_count(eng.model.ctx)
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup)):
            step()
        stream.synchronize()
        eng.check_device("warmup")
        launches_per_step = (B.hsd_launch_count(eng.model.ctx) - launches0) // max(3, args.warmup)
        graph = None
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step()
            for _ in range(3):
                graph.replay()
            stream.synchronize()
    run = (lambda: graph.replay()) if graph is not None else step

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        barrier()
        torch.cuda.cudart().cudaProfilerStart()       # lets `ncu --profile-from-start off` see the timed steps only
        e0.record(stream)
        for _ in range(args.steps):
            run()
        e1.record(stream)
        barrier()
        torch.cuda.cudart().cudaProfilerStop()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    clocks["sampled"] = "timed region"
    if clocks["samples"] < 3:        # a short timed region leaves nvidia-smi nothing to sample: replay longer
        sampler = ClockSampler(uuid)
        with torch.cuda.stream(stream):
            t_end = time.time() + 1.5
            while time.time() < t_end:
                for _ in range(20):
                    run()
                stream.synchronize()
        clocks = sampler.stop()
        clocks["sampled"] = "1.5 s replay of the same step after the timed region"
    if world > 1:
        tt = torch.tensor([ms_total], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_total = float(tt.item())
    ms_step = ms_total / args.steps
    draft_tokens = sum(st["ks"])
    if tree:          # the nodes the device actually packed
        draft_tokens = int(bout["n_rows"].sum().item()) - S
    value = draft_tokens * world / (ms_step * 1e-3)

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
            d_window.copy_(h_win, non_blocking=True)
            eng.dsv_build(d_window, d_dtok, d_doff, d_dsoff, max_q, out=bout)
            eng.verify_tree(bout["q_tokens"], bout["cu_q"], bout["parent"], max_q, T, out=out, log_tau=LOG_TAU_TREE)
            eng.commit_tree(out["accept_len"], out["accept_rows"])
            h_acc.copy_(out["accept_len"], non_blocking=True)
            h_nem.copy_(out["n_emit"], non_blocking=True)
            h_emit.copy_(out["emit_tokens"], non_blocking=True)
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
    e2e = {"value": draft_tokens * world / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": int(h_win.numel() * 4 if tree else h_toks.numel() * 4 + h_cu.numel() * 4),
           "d2h_bytes_per_step": int((h_acc.numel() + h_nem.numel() + h_emit.numel()) * 4 + 16),
           "call": "hsd_verify_regions_host (pinned host buffers; the library replays the step as a CUDA graph it captured "
                   "at the second call of this shape; stream synchronised per step)" if not tree else
                   "hsd_dsv_build + hsd_verify_tree + hsd_kv_commit_tree (eager launches), the window copied in from and "
                   "the results out to pinned host memory on the same stream, synchronised per step"}
    accept_mean = float(np.mean([a / k for a, k in zip(h_acc.numpy().tolist(), st["ks"])]))

    # ---- per-kernel durations (CUDA events around every launch, eager) for the roofline of the top kernel
    peaks, peak_src = load_peaks()
    prof_steps = max(3, min(args.steps, 30))
    with torch.cuda.stream(stream):
        B.hsd_profile_enable(eng.model.ctx, 1)
        for _ in range(prof_steps):
            step()
        stream.synchronize()
        _, prof = B.hsd_profile_read(eng.model.ctx)
        B.hsd_profile_enable(eng.model.ctx, 0)
    ctx_lens = [s.prefix_len for s in st["wl"].seqs]
    work = RF.step_work(cfg, ctx_lens, [k + 1 for k in st["ks"]])
    table = kernel_work_table(cfg, work, T)
    tot_ms = sum(v[0] for v in prof.values()) or 1.0
    kernels = {k: {"ms_per_step": v[0] / prof_steps, "launches_per_step": v[1] / prof_steps,
                   "share": v[0] / tot_ms} for k, v in prof.items()}
    # the dominant kernel class: the largest measured total; classes within 5 % of it count as tied (their order flips
    # from run to run) and the tie goes to the one whose algorithmic roofline time is larger
    cands = [k for k in prof if k in table]
    t_max = max(prof[k][0] for k in cands)

    def roof_time(k):
        fl, nb = table[k]
        return max(fl / (peaks["bf16_tflops_sustained"] * 1e12), nb / (peaks["hbm_gbs"] * 1e9)) * prof[k][1]
    top = max((k for k in cands if prof[k][0] >= 0.95 * t_max), key=roof_time)
    flops, nbytes = table[top]
    dur = prof[top][0] * 1e-3 / prof[top][1]
    bw = peaks["hbm_gbs"] * 1e9
    pk = peaks["bf16_tflops_sustained"] * 1e12
    if flops / pk >= nbytes / bw:
        roof = {"kernel": top, "bound": "tensor", "achieved": flops / dur / 1e12, "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "peak_burst": peaks["bf16_tflops"]}
    else:
        roof = {"kernel": top, "bound": "hbm", "achieved": nbytes / dur / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(top) if args.workload == "region" else None
    roof["peak_source"] = (f"{peak_src} (sustained bf16 figure: kernel timed inside a long step)" if roof["bound"] == "tensor"
                           else f"{peak_src} (STREAM-style copy bandwidth)")
    roof["us_per_launch"] = dur * 1e6
    # the same fraction for every kernel class with a work model (the `roofline` object above is the top one)
    for k, (fl, nb) in table.items():
        if k in prof and prof[k][1] > 0:
            # the LM-head class has one GEMM per step beside a small clearing kernel: its work model is per step
            d_k = prof[k][0] * 1e-3 / (prof_steps if k == "lm_head_argmax" else prof[k][1])
            tensor_k = fl / pk >= nb / bw
            kernels[k]["bound"] = "tensor" if tensor_k else "hbm"
            kernels[k]["roofline_frac"] = (fl / d_k / pk) if tensor_k else (nb / d_k / bw)
    t_roof = RF.roofline_time(work.bytes, work.flops, bw, pk)
    step_roof = {"roofline_us": t_roof * 1e6, "frac": t_roof / (ms_step * 1e-3), "bytes": work.bytes, "flops": work.flops,
                 "bound": "tensor" if work.flops / pk > work.bytes / bw else "hbm"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.workload == "region":
        cpu = cpu_baseline_sample(st["wl"], budget_s=20.0)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOADS[args.workload] + (f" [64 regions only, every draft {args.mixed_k} tokens]"
                                                                   if args.workload == "mixed" and args.mixed_k else ""),
                           "regions_per_gpu": S, "query_rows_per_gpu": T, "draft_tokens_per_gpu": draft_tokens,
                           "context_tokens_per_gpu": int(sum(ctx_lens)), "mean_acceptance_rate": accept_mean,
                           "planted_acceptance_rate": float(np.mean([s.agree_len / s.draft_len for s in st["wl"].seqs])),
                           "l2_policy": "inputs larger than L2: 822 MB of weights are streamed every step",
                           "launch": "CUDA graph replay" if graph is not None else "eager",
                           "sharding": "regions sharded across ranks, no data-path collective"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches_per_step * args.steps),
                "gpu_launches_per_step": int(launches_per_step), "roofline": roof, "step_roofline": step_roof,
                "kernels": kernels, "cpu_baseline": cpu}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------ oracle arm
def cpu_baseline_sample(wl, budget_s=20.0, steps=1, warmup=0):
    """Times the oracle (float32, as it stands) on the two shortest regions of the workload: prefix K/V is
    built first (untimed), then one verify step per region is timed."""
    from oracle import hsd_oracle as O
    weights = I.make_weights(wl.cfg, I.BASE_SEED + 1)
    model = O.Decoder(wl.cfg, weights, np.float32)
    order = sorted(range(len(wl.seqs)), key=lambda i: wl.seqs[i].prefix_len + wl.seqs[i].draft_len)[:2]
    caches, pend, drafts = [], [], []
    for i in order:
        s = wl.seqs[i]
        c = O.CachedSequence(model)
        p = c.prefill(s.prefix_embeds, s.prefix_ids)
        caches.append(c)
        pend.append(p)
        drafts.append(s.rand_tokens[:s.draft_len])        # timing does not depend on the token values
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        O.verify_regions(model, caches, pend, drafts)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
        if sum(times) > budget_s:
            break
    k = int(sum(len(d) for d in drafts))
    t = float(np.mean(times))
    return {"value": k / t, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": f"regions {order} of the workload ({k} draft tokens, contexts "
                      f"{[wl.seqs[i].prefix_len for i in order]}), float32 numpy oracle, prefix K/V prebuilt, "
                      f"{len(times)} timed step(s)", "ms_per_step": t * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = I.region_workload(seed=I.BASE_SEED + 1, cfg=I.DECODER)
    r = cpu_baseline_sample(wl, budget_s=120.0, steps=max(1, args.steps), warmup=max(0, min(args.warmup, 1)))
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "region-level stage (bounded sample: the two shortest regions per step)"},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="region", choices=sorted(WORKLOADS),
                    help="region = the benchmark line; the others time one step of the other configurations")
    ap.add_argument("--mixed-k", type=int, default=0,
                    help="with --workload mixed: the 64 regions alone, every draft this many tokens long (the k sweep)")
    ap.add_argument("--flags", type=int, default=0, help="HSD_FLAG_* bits for the context (debugging / ablations)")
    ap.add_argument("--random-drafts", action="store_true",
                    help="skip the greedy-continuation pass that plants agreement (for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
