"""Region sharding across replicas: the partition, and a world-size-2 run over gloo on CPU in which every rank
verifies only its own regions (the CPU oracle stands in for the per-rank GPU step) and the host-side gather
rebuilds exactly the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import hsd_oracle as O
from paper_2602_12957_b200 import inputs as I
from paper_2602_12957_b200 import shard as SH

CFG = I.ModelConfig(n_layers=1, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=128, vocab=97)


def test_partition_is_a_balanced_exact_cover():
    wl = I.region_workload(cfg=I.small_decoder())
    L = [s.prefix_len for s in wl.seqs]
    k = [s.draft_len for s in wl.seqs]
    for world in (1, 2, 3, 4, 8, 16, 20):
        owned = SH.partition(L, k, world)
        assert len(owned) == world
        flat = sorted(i for o in owned for i in o)
        assert flat == list(range(len(L)))
        assert all(o == sorted(o) for o in owned)
        if world <= 4:
            assert SH.imbalance(L, k, owned) < 1.25
    assert SH.partition(L, k, 2) == SH.partition(L, k, 2)
    with pytest.raises(ValueError):
        SH.partition(L, k[:-1], 2)
    with pytest.raises(ValueError):
        SH.partition(L, k, 0)


def test_cost_model_orders_regions_sensibly():
    assert SH.region_cost(1000, 64) > SH.region_cost(500, 64) > SH.region_cost(500, 8)
    # one row over an empty context: a single attended pair
    assert SH.region_cost(0, 0) == SH.ROW_COST + SH.PAIR_COST


def test_merge_rejects_missing_and_duplicate_regions():
    assert SH.merge_results([{0: "a", 2: "c"}, {1: "b"}], 3) == ["a", "b", "c"]
    with pytest.raises(ValueError):
        SH.merge_results([{0: "a"}, {0: "b"}], 2)
    with pytest.raises(ValueError):
        SH.merge_results([{0: "a"}], 2)


def _verify_subset(wl, weights, which):
    model = O.Decoder(wl.cfg, weights, np.float64)
    out = {}
    for i in which:
        s = wl.seqs[i]
        c = O.CachedSequence(model)
        p = c.prefill(s.prefix_embeds, s.prefix_ids)
        need = min(s.agree_len + 1, s.draft_len)
        g = O.greedy_continuation(c, p, need)
        d = I.plant_draft(g, s.draft_len, s.agree_len, s.rand_tokens, wl.cfg.vocab, False)
        r = O.verify_cached(c, p, d)
        out[i] = (r.accept_len, list(r.emitted))
    return out


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = I.region_workload(seed=5, n_regions=6, prefix_lo=8, prefix_hi=40, draft_mean=6, draft_lo=2, draft_hi=12,
                               cfg=CFG)
        weights = I.make_weights(CFG, 9)
        owned = SH.partition([s.prefix_len for s in wl.seqs], [s.draft_len for s in wl.seqs], world)
        local = _verify_subset(wl, weights, owned[rank])
        merged = SH.gather_results(local, len(wl.seqs))
        # per-rank step time would be reduced with MAX across ranks; check the collective used for that
        t = torch.tensor([float(rank + 1)])
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        q.put((rank, owned, merged, float(t.item())))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_result():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=240) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = I.region_workload(seed=5, n_regions=6, prefix_lo=8, prefix_hi=40, draft_mean=6, draft_lo=2, draft_hi=12, cfg=CFG)
    ref = _verify_subset(wl, I.make_weights(CFG, 9), range(len(wl.seqs)))
    for rank, owned, merged, tmax in got:
        assert sorted(i for o in owned for i in o) == list(range(6)) and all(len(o) > 0 for o in owned)
        assert merged == [ref[i] for i in range(6)]
        assert tmax == float(world)
