"""The benchmark's multi-rank plumbing on CPU (gloo, world_size 2): ranks shard over independent
batches of sequences (no data-path collective), time is the max over ranks, throughput is the sum
of the rows all ranks processed over that time."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    import fork_synth as fs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_info() == (rank, rank, world)
    w = fs.workload("b8")
    seed = bench.shard_seed(w.seed, rank)
    cfg = w.cfg()
    cfg.seed = seed
    row = fs.row_host(cfg, 0, 0, 0)[:64].tolist()            # each rank's inputs differ
    local_ms = 10.0 + 5.0 * rank                               # rank 1 is the slow one
    dist.barrier()
    mx = bench.max_over_ranks(local_ms, torch.device("cpu"))
    value = bench.aggregate(w.B * w.block_len, 7, world, mx)
    gathered = [None] * world
    dist.all_gather_object(gathered, (seed, row))
    if rank == 0:
        out.put((mx, value, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_and_aggregate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    mx, value, gathered = out.get(timeout=240)
    for p in procs:
        p.join(timeout=240)
        assert p.exitcode == 0
    assert mx == 15.0
    assert value == 256 * 7 * 2 / 15e-3
    (s0, r0), (s1, r1) = gathered
    assert s0 != s1 and r0 != r1


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.shard_seed(5, 0) == 5
