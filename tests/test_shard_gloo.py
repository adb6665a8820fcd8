"""Multi-process (gloo, world_size 2 and 3) check of the host logic that shards a batch over GPUs: every user lands
on exactly one rank, the per-rank results reassemble to the single-process result, and timings reduce to the
slowest rank.  The per-rank compute stands in for the single-GPU path and is the CPU oracle here."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lime_oracle as O
from paper_2510_18239_b200 import shard, synth
from tests import lime_helpers as Hh


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload():
    return synth.Workload("shard", B=7, n_min=3, n_max=60, d=16, H=2, ell=4, n_layers=2, C=9, dtype=synth.F32, V=300,
                          zipf_s=1.1, table_std=0.5, link_std=1.0)


def _oracle_logits(wl, inp, users):
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])
    out = [Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg)[0] for b in users]
    return np.concatenate(out) if out else np.zeros(0)


def _rank_main(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = _workload()
        inp = synth.make_inputs(wl, seed=3)                       # every rank draws the same batch, then takes its part
        cands = [wl.C] * wl.B
        parts = shard.partition_users(shard.user_costs(inp["lengths"], cands, wl.ell, wl.n_layers), world)
        lo, hi = parts[rank]
        tok, cnd = shard.shard_slices(inp["lengths"], cands, lo, hi)
        off = O.lengths_to_offsets(inp["lengths"])
        assert (tok.start, tok.stop) == (off[lo], off[hi]) and (cnd.start, cnd.stop) == (lo * wl.C, hi * wl.C)
        local = torch.from_numpy(_oracle_logits(wl, inp, range(lo, hi)))
        counts = [(b - a) * wl.C for a, b in parts]
        full = shard.gather_logits(local, counts)
        slow = shard.max_over_ranks(1.0 + rank)                   # rank r "took" 1 + r seconds
        thr = shard.whole_job_throughput(float(local.numel()), 1.0 + rank)
        ret[rank] = (full.numpy(), slow, thr, parts)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_batch_reassembles_and_times_reduce_to_slowest_rank(world):
    port = _free_port()
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, ret)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    wl = _workload()
    inp = synth.make_inputs(wl, seed=3)
    want = _oracle_logits(wl, inp, range(wl.B))
    for r in range(world):
        full, slow, thr, parts = ret[r]
        assert np.array_equal(full, want)                          # same arithmetic on every rank: exact
        assert slow == float(world)                                # slowest rank
        assert thr == pytest.approx(wl.B * wl.C / float(world))
        assert parts[0][0] == 0 and parts[-1][1] == wl.B
        assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))


def test_partition_is_balanced_contiguous_and_total():
    r = np.random.default_rng(0)
    for world in (1, 2, 4, 8):
        costs = r.integers(1, 1000, size=257)
        parts = shard.partition_users(costs, world)
        assert len(parts) == world and parts[0][0] == 0 and parts[-1][1] == costs.size
        assert all(a <= b for a, b in parts) and all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
        loads = [costs[a:b].sum() for a, b in parts]
        assert max(loads) <= costs.sum() / world + costs.max()     # within one user of the ideal share
    assert shard.partition_users([5, 5], 4)[-1][1] == 2            # fewer users than ranks: some ranks empty
    assert shard.partition_users([], 3) == [(0, 0)] * 3
    assert shard.partition_users([0, 0, 0, 0], 2) == [(0, 2), (2, 4)]
