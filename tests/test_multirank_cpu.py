"""N > 1 host logic on CPU (gloo, world_size 2): the split of a parameter set by whole tensors is a
partition that every rank derives alone, stepping the shards separately gives the bits of the unsplit
set (no data-path collective exists in the method), and the benchmark's max-over-ranks time reduction."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _mini():
    from paper_2601_22101_b200 import workloads as wl
    shapes = [(3, 384), (8, 256), (5, 200), (16, 128), (1, 130), (2, 1024), (7, 384)]
    ts = [wl.TensorSpec(f"t{i}", r, c, 40 + i) for i, (r, c) in enumerate(shapes)]
    return wl.Workload("mini_mr", wl.FP8_E4M3, wl.PER_BLOCK, 128, wl.SCALE_F32, wl.ADAM, wl.SR, lr=1e-3, beta1=0.9,
                       beta2=0.95, eps=1e-8, weight_std=0.02, grad_std=1e-3, steps=3, step_seed=77, tensors=ts)


def _worker(rank: int, world: int, port: int, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle_runner import OracleState
        from paper_2601_22101_b200 import workloads as wl
        w = _mini()
        mine = wl.shard(w, rank, world)
        # every rank derives the same partition alone: gather the ids and check disjoint + complete
        ids = [t.tensor_id for t in mine.tensors]
        gathered = [None] * world
        dist.all_gather_object(gathered, ids)
        flat = [i for g in gathered for i in g]
        assert sorted(flat) == sorted(t.tensor_id for t in w.tensors), "shards must partition the set"
        assert len(set(flat)) == len(flat)
        loads = [sum(t.numel for t in wl.shard(w, r, world).tensors) for r in range(world)]
        assert max(loads) - min(loads) <= max(t.numel for t in w.tensors)
        # step the shard; rank 0 also steps the unsplit set and compares bit for bit
        ora = OracleState(mine, threads=1)
        for step in (1, 2, 3):
            ora.step(step)
        result = {t.tensor_id: (ora.w[i].copy(), ora.scale[i].copy(), ora.m[i].copy(), ora.v[i].copy())
                  for i, t in enumerate(mine.tensors)}
        everyone = [None] * world
        dist.all_gather_object(everyone, result)
        if rank == 0:
            full = OracleState(w, threads=1)
            for step in (1, 2, 3):
                full.step(step)
            merged = {}
            for r in everyone:
                merged.update(r)
            for i, t in enumerate(w.tensors):
                cw, cs, cm, cv = merged[t.tensor_id]
                assert (cw == full.w[i]).all() and (cs.view(np.int32) == full.scale[i].view(np.int32)).all()
                assert (cm.view(np.int32) == full.m[i].view(np.int32)).all()
                assert (cv.view(np.int32) == full.v[i].view(np.int32)).all()
        # the amax exchange of a row-sharded per-tensor step: an integer MAX over the bit patterns of
        # non-negative binary32 values is their floating-point maximum
        mine_amax = torch.tensor([0.0, 1e-30, 0.5 + rank, 3.0 - rank, 447.9999], dtype=torch.float32)
        bits = mine_amax.view(torch.int32).clone()
        dist.all_reduce(bits, op=dist.ReduceOp.MAX)
        expect = torch.tensor([0.0, 1e-30, 0.5 + world - 1, 3.0, 447.9999], dtype=torch.float32)
        assert torch.equal(bits.view(torch.float32), expect)
        # the benchmark's time reduction: max over ranks
        t = torch.tensor([10.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == 10.0 + world - 1
        dist.barrier()
        q.put((rank, "ok"))
    except Exception as e:  # report instead of hanging the peer
        q.put((rank, f"{type(e).__name__}: {e}"))
    finally:
        dist.destroy_process_group()


def test_shard_partition_and_invariance_two_ranks():
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
    assert sorted(got) == [(0, "ok"), (1, "ok")], got


def test_shard_and_replicate_host_logic():
    from paper_2601_22101_b200 import workloads as wl
    w = wl.c5()
    parts = [wl.shard(w, r, 8) for r in range(8)]
    assert sum(len(p.tensors) for p in parts) == len(w.tensors)
    assert sum(p.numel for p in parts) == w.numel
    loads = [p.numel for p in parts]
    assert max(loads) - min(loads) <= max(t.numel for t in w.tensors)
    with pytest.raises(ValueError):
        wl.shard(w, 8, 8)
    r = wl.replicate(wl.c2(), 3)
    assert r.numel == 3 * wl.c2().numel and len({t.tensor_id for t in r.tensors}) == len(r.tensors)
