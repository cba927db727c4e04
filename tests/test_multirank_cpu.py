"""World-size-2 checks of the multi-rank host logic, on CPU with gloo: head
sharding is a partition, shards are independent (no exchange needed), and the
benchmark's max-over-ranks / aggregate arithmetic."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        import oracle
        import workloads
        w = workloads.small_structured(H=5, d=64, grid=(2, 8, 20), block=64, sparsity=0.6, cfg_id=55)
        qq, kk, vv = workloads.structured_qkv(w)
        mine = list(workloads.shard_heads(w.H, world, rank))
        # each rank works on its heads only: selection + attention need nothing from the other rank
        idx, cnt = oracle.select(qq[0, mine], kk[0, mine], w.block, w.topk)
        out, _ = oracle.attention(qq[0, mine], kk[0, mine], vv[0, mine], idx, cnt, w.block)
        gathered = [None] * world
        dist.all_gather_object(gathered, (mine, idx, out))
        # timing reduction: the slowest rank defines the step time
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")
        agg = bench.aggregate_throughput(2.0e12, ms, world)
        # head-sharded mode of the benchmark: every rank counts the kept FLOPs of its own heads, the job's
        # throughput is their sum over the slowest rank's time
        w_mine = w.with_heads(len(mine))
        strong = bench.sharded_throughput(float(bench.kept_flops(w_mine, idx, cnt)), ms, "cpu")
        if rank == 0:
            heads = sum((g[0] for g in gathered), [])
            full_idx, full_cnt = oracle.select(qq[0], kk[0], w.block, w.topk)
            full_out, _ = oracle.attention(qq[0], kk[0], vv[0], full_idx, full_cnt, w.block)
            ok_part = sorted(heads) == list(range(w.H)) and len(heads) == w.H
            ok_idx = torch.equal(torch.cat([g[1] for g in gathered]), full_idx)
            ok_out = torch.equal(torch.cat([g[2] for g in gathered]), full_out)
            full_flops = bench.kept_flops(w, full_idx, full_cnt)
            ok_strong = abs(strong - full_flops / (ms * 1e-3) / 1e12) <= 1e-9 * max(1.0, strong)
            q.put((ok_part, ok_idx, ok_out, ms, agg, ok_strong))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_heads_without_exchange():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = q.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ok_part, ok_idx, ok_out, ms, agg, ok_strong = res
    assert ok_part and ok_idx and ok_out and ok_strong
    assert ms == 15.0
    assert abs(agg - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9


def test_shard_heads_is_a_balanced_partition():
    import workloads
    for H in (1, 5, 12, 40):
        for world in (1, 2, 3, 8):
            shards = [list(workloads.shard_heads(H, world, r)) for r in range(world)]
            assert sum(shards, []) == list(range(H))
            sizes = [len(s) for s in shards]
            assert max(sizes) - min(sizes) <= 1
