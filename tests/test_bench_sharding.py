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


def _vp_worker(rank, world, port, q):
    import torch
    import torch.distributed as dist
    from paper_2609_39859_b200.binding import gather_rank_major, vocab_shards
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        shards = vocab_shards(126464, world, 2)
        off, n = shards[rank]
        mine = torch.full((3, 5, 4), float(rank), dtype=torch.float32)
        mine[0, 0, 3] = off
        got = gather_rank_major(mine)
        ok = got.shape == (world, 3, 5, 4) and all(float(got[r, 1, 1, 0]) == r and int(got[r, 0, 0, 3]) == shards[r][0]
                                                    for r in range(world))
        q.put((rank, bool(ok)))
    finally:
        dist.destroy_process_group()


def test_vocab_shards_and_rank_major_gather_with_two_gloo_ranks():
    """Host side of the vocabulary-parallel step: slices cover the vocabulary, start on 16-byte
    boundaries and ascend with the rank; the gather returns the ranks' buffers in rank order."""
    import multiprocessing as mp
    import socket
    from paper_2609_39859_b200.binding import vocab_shards
    for V, n, es in ((126464, 8, 2), (152064, 4, 2), (126464, 3, 4), (1000, 3, 2), (7, 4, 4)):
        sh = vocab_shards(V, n, es)
        assert sum(l for _, l in sh) == V and sh[0][0] == 0
        for (o0, l0), (o1, _) in zip(sh, sh[1:]):
            assert o1 == o0 + l0 or (l0 == 0 and o1 == V)
        assert all((o * es) % 16 == 0 for o, l in sh if l > 0)
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_vp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == [(0, True), (1, True)]
