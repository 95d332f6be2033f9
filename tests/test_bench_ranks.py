"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, no GPU.  The verification step
shards by sequence (replicas, no data-path collective); what the ranks exchange is only the
timing / token bookkeeping checked here."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2601_00644_b200 import workloads as wl
    shape = bench.shard_for_rank(wl.CONFIGS["tiny"], rank)
    inp = wl.make_inputs(shape, device="cpu")
    # every rank reports its own time and token count; rank r is the slower the larger r is
    total_ms, e2e_s, tokens = bench.reduce_over_ranks(10.0 + rank, 0.5 * (rank + 1), 100 + 7 * rank)
    out.put((rank, shape.index, int(inp.seeds[0]), total_ms, e2e_s, tokens))
    dist.destroy_process_group()


def test_two_ranks_take_max_time_and_sum_tokens_with_distinct_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, idx0, seed0, ms0, e0, tok0), (r1, idx1, seed1, ms1, e1, tok1) = res
    assert idx0 != idx1 and seed0 != seed1          # replicas verify different batches
    assert ms0 == ms1 == 11.0                       # slowest rank
    assert e0 == e1 == 1.0
    assert tok0 == tok1 == 207.0                    # whole-job tokens


def test_single_process_is_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.0, 0.25, 11) == (3.0, 0.25, 11.0)
