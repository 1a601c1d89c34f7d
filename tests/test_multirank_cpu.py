"""World-size-2 checks on CPU (gloo): the pieces of the N > 1 path that need no GPU.
The operator has no exchange step, so ranks only agree on (a) which global KV heads each one
owns -- windows are assigned by global head index, Eq. (fwa_global_head) -- and (b) the timing
reduction the benchmark uses (slowest rank)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
import paper_2609_32704_b200 as cowa
from oracle import cowa_oracle as orc

WORLD = 2


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        # (a) tensor-parallel head sharding: rank r owns global heads [r*H/W, (r+1)*H/W)
        Nk, Hkv, sink, near, blk = 3000, 8, 16, 200, 64
        local = Hkv // WORLD
        mine = cowa.cowa_default_windows(Nk, Hkv, rank * local, local, sink, near)
        p = cowa.make_params(sink=sink, local=near, block=blk, hkv_global=Hkv, hkv_offset=rank * local)
        sched = cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nk, Nk, local, p)
        gathered = [None] * WORLD
        dist.all_gather_object(gathered, (mine, sched))
        # (b) timing reduction
        slowest = bench.max_over_ranks(10.0 + rank, WORLD)
        bench.barrier(WORLD)
        if rank == 0:
            windows = [w for g in gathered for w in g[0]]
            ok_w = windows == orc.default_windows(Nk, Hkv, sink, near)
            # each rank's schedule equals the single-rank schedule of the same global heads
            full = cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nk, Nk, Hkv,
                                           cowa.make_params(sink=sink, local=near, block=blk))
            def by_head(stream, nheads):
                recs, pos = {}, 0
                while pos < len(stream):
                    h, i, n = stream[pos:pos + 3]
                    recs.setdefault(h, []).append(tuple(stream[pos + 1:pos + 3 + 2 * n]))
                    pos += 3 + 2 * n
                return [recs[h] for h in range(nheads)]
            glob = by_head(full, Hkv)
            ok_s = all(by_head(gathered[r][1], local) == glob[r * local:(r + 1) * local] for r in range(WORLD))
            out.put((ok_w, ok_s, slowest))
        else:
            out.put(("rank1", slowest))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_global_heads_and_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, port, out)) for r in range(WORLD)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(WORLD)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    r0 = [r for r in results if r[0] != "rank1"][0]
    r1 = [r for r in results if r[0] == "rank1"][0]
    assert r0[0] and r0[1]
    assert r0[2] == 11.0 and r1[1] == 11.0


def _tp_worker(rank, world, port, out):
    """bench.py --tp-replica under N processes: which TP=8 shards each process times, and the reduction of the
    per-phase slowest shard over the processes (made-up latencies stand in for the GPU timings)."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shards = bench.tp_shards(rank, world, 8)
        # shard r "takes" 10 + r ms forward and 30 - r ms backward at one length, so the slowest forward shard is
        # 7 and the slowest backward shard is 0, whoever owns them
        row = {"T": 4096, "cowa_fwd_ms": max([10.0 + r for r in shards], default=0.0),
               "cowa_bwd_ms": max([30.0 - r for r in shards], default=0.0)}
        reduced = bench.reduce_worst([row], world)
        gathered = [None] * world
        dist.all_gather_object(gathered, shards)
        out.put((rank, gathered, reduced))
    finally:
        dist.destroy_process_group()


def _run_tp(world):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_tp_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return results


def test_tp_replica_shard_assignment_and_worst_shard_reduction():
    for world in (2, 8):
        for rank, gathered, reduced in _run_tp(world):
            # every shard of the TP=8 group is timed by exactly one process; with 8 processes one each
            assert sorted(s for g in gathered for s in g) == list(range(8))
            assert gathered[rank] == list(range(rank, 8, world))
            if world == 8:
                assert all(len(g) == 1 for g in gathered)
            # every process ends up with the group's latency: the slowest shard per phase
            assert reduced == [{"T": 4096, "cowa_bwd_ms": 30.0, "cowa_fwd_ms": 17.0}]
    assert bench.tp_shards(9, 16, 8) == []  # surplus processes own nothing
