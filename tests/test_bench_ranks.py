"""The only multi-rank logic of the path: replicas combine their timings (max) and token counts (sum).  Run as two
gloo ranks on the CPU."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms, tokens = bench.combine_ranks(10.0 + 5.0 * rank, 100.0 + rank, world, device="cpu")
        out[rank] = (ms, tokens, bench.throughput(ms, tokens))
    finally:
        torch.distributed.destroy_process_group()


def test_two_replicas_combine_max_time_and_sum_tokens():
    world = 2
    port = 29500 + os.getpid() % 1000
    with mp.Manager() as man:
        out = man.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in range(world):
        ms, tokens, value = res[r]
        assert ms == 15.0 and tokens == 201.0
        assert abs(value - 201.0 / 0.015) < 1e-9


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.combine_ranks(3.0, 7.0, 1) == (3.0, 7.0)
