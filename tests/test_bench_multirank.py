"""The N > 1 path of bench.py is "replicas only": ranks share nothing but the timing reduction.  Two gloo ranks
on the CPU check that reduction and the whole-job aggregate."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    dec = bench.aggregate("decode", 1, ms / 100, world)            # 100 steps each
    pre = bench.aggregate("prefill", 512, ms / 100, world)
    out[rank] = (ms, dec[1], dec[3], pre[1], pre[3])
    torch.distributed.barrier()
    torch.distributed.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, 29500 + os.getpid() % 1000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, dec, dec_hib, pre, pre_hib = res[0]
    assert ms == 15.0
    assert abs(dec - 0.15e3 / 2) < 1e-9 and dec_hib is False       # us per token over 2 replicas' tokens
    assert abs(pre - 512 * 2 / 0.15e-3) < 1e-3 and pre_hib is True  # tokens per second of the whole job


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
